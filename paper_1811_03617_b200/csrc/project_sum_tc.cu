// Projection fused with the N-way compressed-domain sum (Eq. 3 + Eq. 4) on the 5th-generation
// tensor cores (tcgen05, kind::tf32, accumulators in tensor memory).
//
//   s_sum[i] = sum_n  Ut_l (x_{n,i} - mu_l / N)
//
// At k = 16 / 32 the projection needs 8 / 16 flop per input byte, beyond what the FP32 pipe
// sustains at HBM speed, while it is a dense tall-skinny contraction:  a tile of 128 slices is
// the M = 128 side, the (node, slice entry) pairs are the contraction, the k outputs are N.
// Plain TF32 would miss the 1e-5 parity bar, so every product is split into three TF32 products
// with fp32 accumulation:      x u ~= x_hi u_hi + x_hi u_lo + x_lo u_hi
// (hi = the value cut to TF32 precision, lo = the exact remainder), issued as
//      D1[:, 0:2k] += A_hi [U_hi | U_lo]       D2[:, 0:k] += A_lo U_hi       s_n = D1[:, :k] + D1[:, k:] + D2
// The tensor core's fp32 accumulator rounds toward zero, so a long accumulation chain drifts (the
// measured relative error grew as 1.2e-6 x the number of nodes chained).  One node's d entries are
// therefore the longest chain: each node's compressed tile is read back from tensor memory and the
// sum over the nodes (Eq. 4) is carried in registers with round-to-nearest adds.
//
// One persistent CTA per SM, warp-specialised (G = 3 converter groups of 4 warps):
//   warps 0..4G-1  converters: thread <-> slice (<-> tensor-memory lane).  Read the 32 entries of the own
//               slice (the swizzle makes these per-row reads bank-conflict free), subtract mu / N
//               (exactly as Eq. 3 orders it), split into hi / lo and store both into a tensor-memory
//               A buffer (tcgen05.st); five A buffers rotate, sub-chunk c goes to warp group c % G.
//               A stage goes back to the producer only after its values were consumed (after the
//               tcgen05.st and its wait): released earlier, the next load overwrote data in flight.
//   warp 4G     producer: one thread issues one tiled TMA load (cp.async.bulk.tensor.2d, 128-byte
//               swizzle) per 128 slices x 32 entries (16 KB) into a ring of shared-memory stages;
//               one tensor map per (node, layer) makes the rows past a layer's last slice read as 0
//   warps 4G+1, 4G+2  issue tcgen05.mma (A from tensor memory, [U_hi | U_lo] from shared memory in the
//               canonical K-major 128-byte-swizzled layout): the first the x_hi products, the second
//               the x_lo products, into separate accumulators -- one thread issues at most one MMA per
//               ~50-70 clocks, more than these small MMAs take to execute.  Their loops are warp-uniform
//               with one elected lane issuing; they commit to the mbarriers that recycle the A buffers
//               and publish the accumulators
//   groups 0, 1 after each node: tcgen05.ld of that node's accumulator (two rotate), half of the k
//               columns per group, hi + lo parts added into the running sum in registers; after the
//               last node 128-bit stores.  Quantizing variant: group 0 alone reads back, all k columns of a
//               slice in one thread (the norm needs them all), and converts nothing; it parks the vector in
//               shared memory, returns the accumulator, and applies gvq_quantize's arithmetic eight
//               coordinates at a time before the vector enters the sum (registers: 128 per thread).
// Work is dealt in (tile, node) units, the same number to every CTA, as contiguous runs: a CTA shares
// at most its first and its last tile with a neighbour.  Of the two CTAs of a shared tile the one that
// finishes second (a ticket per tile) adds (lower nodes' partial) + (upper nodes' partial) in that order
// and writes s_sum, so the result does not depend on timing.
// The raw gradient crosses shared memory once (written by TMA, read by the converters);
// the tensor core reads A from tensor memory.  Every wait on an mbarrier is bounded: when a limit
// is hit the CTA records an error word, drains its copies, frees its tensor memory and returns.
#include "gvq_internal.h"
#include "quantizer.cuh"
#include "sm100_ptx.cuh"

namespace gvq {
namespace {

constexpr int TM = kProjectTcRows;   // slices per tile (MMA M)
constexpr int NS = 9;                // shared-memory stages of 16 KB
// Converter groups: three, of 4 warps each (one per tensor-memory lane quarter).  Sub-chunk c normally goes to
// group c % 3; in the quantizing variant group 0 runs the quantizer instead and groups 1 and 2 take turns.
__host__ __device__ constexpr int groups_of(bool) { return 3; }
__host__ __device__ constexpr int threads_of(bool quant) { return (4 * groups_of(quant) + 3) * 32; }   // + producer + two MMA issuers
constexpr int NABUF = 5;             // tensor-memory A buffers of 64 columns (32 hi + 32 lo)
constexpr uint32_t D_STRIDE = 96;    // columns per node accumulator set: D1 [0, 2 KP), D2 [64, 64 + KP)
constexpr uint32_t D2_OFF = 64;
constexpr uint32_t A_COL0 = 192;     // two accumulator sets live in columns [0, 192), A buffers above
constexpr uint32_t TMEM_COLS = 512;

struct TcParams {
    int d, n_tiles, n_nodes, mean_div;
    const int32_t *tile_layer, *tile_row0;
    const int64_t *layer_off, *layer_soff;
    const int32_t *layer_S;
    const float *Ut, *mu;
    float *s_sum;
    int32_t *error_word;
    const CUtensorMap *tmaps;  // [slot][layer]: 2-D view (d entries x S_l slices) of one layer of one node
    int n_layers;
    int slot[GVQ_MAX_NODES];   // which slot holds node n's maps
    NodePtrs<float> s_nodes;   // optional per-node outputs (all NULL when not wanted)
    // quantizing variant: every node's compressed vector is quantized (gvq_quantize's definition) and the
    // dequantised vectors are summed; q_nodes / norms optionally receive what each node would transmit
    int levels;
    uint64_t seed;
    NodePtrs<int8_t> q_nodes;
    NodePtrs<float> norms;
    double *monitor;           // [n_layers][2][n_nodes]: sum |x - mu / N|^2, sum |s_n|^2 (MON variant)
    int32_t ustart[kMaxPartitionCtas + 1];   // CTA b works on units [ustart[b], ustart[b + 1])
    float *partial;            // [2 * gridDim][128][KP] sums over a node range of a tile shared with a neighbour CTA
    int32_t *tile_counter;     // [n_tiles] arrival tickets of such tiles, zero between launches
    int wait_kcycles;          // limit of every bounded wait, in units of 1024 clocks
    int drop_last_load;        // test hook: CTA 0 leaves out the very last load of its run, so a wait runs out
    int64_t slice_base;        // added to a slice's index where it keys the quantizer's hash (contexts over a part of a layout)
};

using namespace ptx;

struct Smem {
    // offsets (bytes) into dynamic shared memory, which is aligned to 1024
    uint32_t b, mu, stage, bars, sq, total;
};
__host__ __device__ inline Smem smem_layout(int d, int kp, bool quant = false)
{
    Smem s;
    s.b = 0;                                            // [d / 32][2 kp rows][128 B]   swizzled
    s.stage = s.b + (uint32_t)d * 2 * kp * 4;           // [NS][128 rows][128 B]        swizzled, 1024-aligned
    s.mu = s.stage + (uint32_t)NS * TM * 128;           // [d] floats
    s.bars = (s.mu + (uint32_t)d * 4 + 15) & ~15u;
    s.sq = s.bars + 512 + 2 * GVQ_MAX_NODES * 4;      // 33 mbarriers, the tensor-memory slot, two flag words; monitor sums
    s.total = s.sq + (quant ? (uint32_t)kp * TM * 4 : 0);   // quantizing variant: [kp][128 slices] one node's compressed tile
    return s;
}

// KP: compressed length (16 or 32) = N of the x_lo MMA; the x_hi MMA has N = 2 KP.
// QUANT: quantize each node's vector before it enters the sum.
// MON: also accumulate, per layer and node, sum |x - mu / N|^2 over the slices (by the converter threads, which hold
// the centred entries anyway) and sum |s_n|^2 (by the threads that read the accumulators back): the two terms of
// Eq. 7's local compression loss, |x_c - U s|^2 = |x_c|^2 - |s|^2 for a basis with orthonormal columns.
template <int KP, bool QUANT, bool MON>
__global__ void __launch_bounds__(threads_of(QUANT), 1) project_sum_tc_kernel(const __grid_constant__ TcParams prm)
{
    constexpr int NPAR = groups_of(QUANT), NCONV = 4 * NPAR;
    // Warps that read the accumulators back: groups 0 and 1, half of the k columns each -- or, when
    // quantizing, group 0 alone with all k columns of its slice in one thread (the norm needs them all),
    // while groups 1 and 2 convert.
    constexpr int NDR = QUANT ? 4 : 8;
    constexpr int COLS = QUANT ? KP : KP / 2;
    extern __shared__ unsigned char smem_raw[];
    // the swizzled basis tiles need a 1024-byte aligned base
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int d = prm.d;
    const int SUBS = d / 32;                     // 32-entry sub-chunks per slice (even)
    const Smem L = smem_layout(d, KP, QUANT);
    float *muN = reinterpret_cast<float *>(smem + L.mu);
    unsigned char *stage0 = smem + L.stage;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint64_t *full = bars;                 // [NS]     copies landed             (producer -> converters)
    uint64_t *empty = bars + NS;           // [NS]     stage read                (converters -> producer)
    uint64_t *a_full = bars + 2 * NS;      // [NABUF]  A buffer written          (converters -> MMA)
    uint64_t *a_empty = a_full + NABUF;    // [NABUF]  A buffer consumed         (MMA -> converters)
    uint64_t *d_full = a_empty + NABUF;    // [2]      accumulator complete      (MMA -> epilogue)
    uint64_t *d_empty = d_full + 2;        // [2]      accumulator drained       (epilogue -> MMA)
    uint64_t *b_ready = d_empty + 2;       // [1]      basis of the layer staged (converters -> MMA)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(b_ready + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    float *mon_s = reinterpret_cast<float *>(smem + L.bars + 512);   // [2][GVQ_MAX_NODES] of the current layer (MON)
    // QUANT (never together with MON): the (seed, node) half of the quantizer's hash for every node, in the same place
    uint64_t *node_keys = reinterpret_cast<uint64_t *>(smem + L.bars + 512);   // [GVQ_MAX_NODES]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x;
    // Work is dealt in units of (tile, node): CTA b takes a contiguous run of them, so its first and last
    // tile may be shared with a neighbour (each then sums a node range and the last to finish adds the
    // pieces).  The runs come from the host, balanced by a cost model that charges a run for every layer it
    // touches (the pipeline is drained and the basis staged at each change of layer).
    auto unit_start = [&](long long b) { return (long long)prm.ustart[b]; };
    auto cta_of_unit = [&](long long u) {   // the last CTA whose run starts at or before unit u and is not empty there
        int lo = 0, hi = G - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if ((long long)prm.ustart[mid] <= u) lo = mid; else hi = mid - 1;
        }
        return (long long)lo;
    };
    const long long u0 = unit_start(blockIdx.x), u1 = unit_start(blockIdx.x + 1);
    const int t_begin = (int)(u0 / prm.n_nodes);
    const int t_end = u1 > u0 ? (int)((u1 - 1) / prm.n_nodes) + 1 : t_begin;
    // nodes [node_lo(tile), node_hi(tile)) of a tile belong to this CTA
    auto node_lo = [&](int tile) { return tile == t_begin ? (int)(u0 - (long long)tile * prm.n_nodes) : 0; };
    auto node_hi = [&](int tile) { return tile == t_end - 1 ? (int)(u1 - (long long)tile * prm.n_nodes) : prm.n_nodes; };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 4); }
        for (int i = 0; i < NABUF; ++i) { mbar_init(a_full + i, 4); mbar_init(a_empty + i, 2); }
        for (int i = 0; i < 2; ++i) { mbar_init(d_full + i, 2); mbar_init(d_empty + i, NDR); }
        mbar_init(b_ready, NCONV);
        *abort_flag = 0;
        const_cast<int *>(abort_flag)[2] = prm.wait_kcycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if constexpr (QUANT) {
        if ((int)threadIdx.x < prm.n_nodes) node_keys[threadIdx.x] = quant::node_key(prm.seed, threadIdx.x);
    }
    if (warp == NCONV + 1) {  // the first MMA warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;
    // The set-up above overlaps the tail of the previous kernel of the stream (normally the decompression of the
    // previous step); from here on this kernel reads and writes global memory.
    launch_dependents();
    grid_dependency_wait();

    if (warp == NCONV) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t issued = 0, s = 0, ph = 0;   // loads issued; the next one's stage and the parity of its use count
            for (int tile = t_begin; tile < t_end && !failed; ++tile) {
                const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile];
                for (int n = node_lo(tile); n < node_hi(tile) && !failed; ++n) {
                    const CUtensorMap *tm = prm.tmaps + (size_t)prm.slot[n] * prm.n_layers + layer;
                    for (int u = 0; u < SUBS; ++u, ++issued, s = (s + 1 == NS ? 0 : s + 1), ph ^= (s == 0)) {
                        if (!mbar_wait(empty + s, ph ^ 1, abort_flag)) { failed = true; break; }
                        // test hook: the last load of CTA 0's run is left out, so that the converters' wait for
                        // it runs out and the give-up path is taken (nothing faults: a wait simply ends)
                        if (prm.drop_last_load && blockIdx.x == 0 && tile == t_end - 1 && n == node_hi(tile) - 1 && u == SUBS - 1)
                            continue;
                        mbar_arrive_expect_tx(full + s, TM * 128);
                        tma_load_2d(stage0 + (size_t)s * TM * 128, tm, u * 32, row0, full + s);
                    }
                }
            }
            if (failed) {
                // give the copies already in flight a bounded chance to land before the CTA exits
                for (uint32_t i = issued > NS ? issued - NS : 0; i < issued; ++i)
                    for (int it = 0; it < 100000 && !mbar_try_wait(full + i % NS, (i / NS) & 1); ++it) {}
            }
        }
        failed = __shfl_sync(0xffffffffu, failed, 0);
    } else if (warp >= NCONV + 1) {
        // ------------------------------------------------------------------ MMA issuers
        // A single thread cannot issue tcgen05.mma faster than one per ~50-70 clocks, whatever its size,
        // while these small MMAs execute in 32 / 16 clocks.  Two warps therefore issue independently into
        // separate accumulators: issuer 0 the products with x_hi (N = 2 KP), issuer 1 those with x_lo (N = KP).
        const int which = warp - (NCONV + 1);
        const uint32_t idesc = which == 0 ? make_idesc(2 * KP) : make_idesc(KP);
        const uint64_t bd0 = make_b_desc(smem_u32(smem + L.b));
        const uint32_t bd0_lo = (uint32_t)bd0, bd0_hi = (uint32_t)(bd0 >> 32);
        // The whole warp walks the loop (waits included) so that control flow stays uniform; one elected
        // lane issues.
        uint32_t m = 0, layers_seen = 0;   // (tile, node) and layer-change counters
        uint32_t ab = 0, ab_par = 0;       // the next sub-chunk's A buffer and the parity of its use count
        int cur_layer = -1;
        for (int tile = t_begin; tile < t_end && !failed; ++tile) {
            const int layer = prm.tile_layer[tile];
            if (layer != cur_layer) {
                bool ok = mbar_wait(b_ready, layers_seen & 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                ++layers_seen;
                cur_layer = layer;
            }
            for (int n = node_lo(tile); n < node_hi(tile) && !failed; ++n, ++m) {
                const uint32_t db = m & 1;
                bool ok = mbar_wait(d_empty + db, ((m >> 1) & 1) ^ 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + db * D_STRIDE + (which ? D2_OFF : 0);
                for (int cc = 0; cc < SUBS; ++cc, ab = (ab + 1 == NABUF ? 0 : ab + 1), ab_par ^= (ab == 0)) {   // cc: which 32 entries of the slice
                    ok = mbar_wait(a_full + ab, ab_par, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t a_op = tmem_base + A_COL0 + ab * 64 + (which ? 32 : 0);
                    const uint32_t bd_lo = bd0_lo + (uint32_t)cc * (2 * KP * 128 / 16);   // 16-byte units
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)   // 8 entries (32 bytes of the swizzled row) per step
                            tc_mma_tf32_ts(d_tmem, a_op + kk * 8, bd_lo + kk * 2, bd0_hi, idesc, kk == 0 ? (uint32_t)cc : 1u);
                        tc_commit(a_empty + ab);
                        if (cc == SUBS - 1) tc_commit(d_full + db);
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ converters + epilogue
        const int q = warp & 3, h = warp >> 2;       // lane quarter, converter group
        const bool drainer = QUANT ? h == 0 : h < 2;
        const int col0 = QUANT ? 0 : h * (KP / 2);    // first of this thread's COLS columns
        const uint32_t lane_base = (uint32_t)(32 * q) << 16;
        const int ctid = threadIdx.x;                 // 0 .. 255 among the converter warps
        uint32_t m = 0;                               // (tile, node) counter
        // This group's share of the sub-chunks: every ST-th one, counted through the CTA's whole run (ST groups
        // convert: all three, or groups 1 and 2 when group 0 runs the quantizer).  Its stage, its A buffer and the
        // parities to wait for are stepped along with it instead of being derived from a running count.
        constexpr int ST = QUANT ? 2 : NPAR;
        const bool converts = !QUANT || h > 0;
        const int gi = QUANT ? h - 1 : h;             // index among the converting groups
        int cc_next = gi;                             // the group's next sub-chunk, counted from the current node's first
        uint32_t s = (uint32_t)(converts ? gi : 0) % NS, s_par = 0;
        uint32_t ab = (uint32_t)(converts ? gi : 0) % NABUF, ab_par = 1;
        int cur_layer = -1;
        // Adds node m's compressed tile (hi + lo columns of its accumulator) to the running sum and
        // hands the accumulator back.  This thread owns columns [h * KP / 2, (h + 1) * KP / 2) of slice r.
        auto drain = [&](uint32_t mm, float (&acc)[COLS], float *sn_row, int node, int64_t gslice, bool live) -> bool {
            const uint32_t db = mm & 1;
            bool ok = mbar_wait(d_full + db, (mm >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) return false;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + lane_base + db * D_STRIDE + col0;
            if constexpr (QUANT) {
                // The node's k coordinates of this thread's slice: summed from the three accumulator parts,
                // parked in shared memory (a column of its own per thread, no one else reads it) so that the
                // accumulator can go back to the tensor core at once, and squared for the norm -- coordinate j
                // together with j + k / 2, the first level of the norm's butterfly.
                float *mine = reinterpret_cast<float *>(smem + L.sq) + (32 * q + lane);
                float t[KP / 2];
#pragma unroll
                for (int v = 0; v < KP / 16; ++v) {
                    float lo8[8];
                    {
                        float a[8], b[8], e[8];   // x_hi u_hi, x_hi u_lo, x_lo u_hi
                        tmem_ld8x3_wait(d_tmem + v * 8, d_tmem + KP + v * 8, d_tmem + D2_OFF + v * 8, a, b, e);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            lo8[i] = a[i] + (b[i] + e[i]);
                            mine[(v * 8 + i) * TM] = lo8[i];
                        }
                    }
                    float a[8], b[8], e[8];
                    tmem_ld8x3_wait(d_tmem + KP / 2 + v * 8, d_tmem + KP + KP / 2 + v * 8, d_tmem + D2_OFF + KP / 2 + v * 8, a, b, e);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float hi = a[i] + (b[i] + e[i]);
                        mine[(KP / 2 + v * 8 + i) * TM] = hi;
                        t[v * 8 + i] = __fadd_rn(__fmul_rn(lo8[i], lo8[i]), __fmul_rn(hi, hi));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d_empty + db);
                const float norm = quant::norm_from_first_level<KP / 2>(t);
                // gvq_quantize's arithmetic, eight coordinates at a time; the dequantised vector enters the running sum
                const quant::BucketKeys keys = quant::bucket_keys(norm, prm.levels, node_keys[node], gslice + prm.slice_base);
                int8_t *qn = live ? prm.q_nodes.p[node] : nullptr;
#pragma unroll
                for (int c8 = 0; c8 < KP / 8; ++c8) {
                    float v8[8], dq[8];
                    uint32_t packed[2];
#pragma unroll
                    for (int i = 0; i < 8; ++i) { v8[i] = mine[(c8 * 8 + i) * TM]; dq[i] = 0.0f; }
                    if (qn) {   // the integer codes are formed only when somebody wants them
                        quant::quantize_columns<8, true>(v8, c8 * 8, keys, packed, dq);
                        *reinterpret_cast<uint2 *>(qn + gslice * KP + c8 * 8) = make_uint2(packed[0], packed[1]);
                    } else {
                        quant::quantize_columns<8, false>(v8, c8 * 8, keys, packed, dq);
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[c8 * 8 + i] += dq[i];
                    if (sn_row) {
                        *reinterpret_cast<float4 *>(sn_row + c8 * 8) = make_float4(v8[0], v8[1], v8[2], v8[3]);
                        *reinterpret_cast<float4 *>(sn_row + c8 * 8 + 4) = make_float4(v8[4], v8[5], v8[6], v8[7]);
                    }
                }
                if (live) {
                    float *nn = prm.norms.p[node];
                    if (nn) nn[gslice] = norm;
                }
                return true;
            } else {
                float sn[COLS];
#pragma unroll
                for (int v = 0; v < COLS / 8; ++v) {
                    float a[8], b[8], e[8];   // x_hi u_hi, x_hi u_lo, x_lo u_hi
                    tmem_ld8x3_wait(d_tmem + v * 8, d_tmem + KP + v * 8, d_tmem + D2_OFF + v * 8, a, b, e);
#pragma unroll
                    for (int i = 0; i < 8; ++i) sn[v * 8 + i] = a[i] + (b[i] + e[i]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d_empty + db);
                if constexpr (MON) {
                    float p2 = 0.0f;
#pragma unroll
                    for (int i = 0; i < COLS; ++i) p2 = fmaf(sn[i], sn[i], p2);
                    if (!live) p2 = 0.0f;
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1) p2 += __shfl_xor_sync(0xffffffffu, p2, o);
                    if (lane == 0) atomicAdd(mon_s + GVQ_MAX_NODES + node, p2);
                }
                if (sn_row) {
#pragma unroll
                    for (int v = 0; v < COLS / 4; ++v)
                        *reinterpret_cast<float4 *>(sn_row + v * 4) =
                            make_float4(sn[4 * v], sn[4 * v + 1], sn[4 * v + 2], sn[4 * v + 3]);
                }
#pragma unroll
                for (int i = 0; i < COLS; ++i) acc[i] += sn[i];
                return true;
            }
        };
        // Monitor sums of the layer just finished go to global memory (between two barriers of the converter warps)
        auto flush_monitor = [&](int layer_done) {
            if (ctid < 2 * GVQ_MAX_NODES) {
                const int which = ctid / GVQ_MAX_NODES, node = ctid % GVQ_MAX_NODES;
                const float v = mon_s[ctid];
                mon_s[ctid] = 0.0f;
                if (layer_done >= 0 && node < prm.n_nodes && v != 0.0f)
                    atomicAdd(prm.monitor + ((size_t)layer_done * 2 + which) * prm.n_nodes + node, (double)v);
            }
        };
        float e2 = 0.0f;   // this thread's share of |x - mu / N|^2 of the current node
        const float2 neg1 = make_float2(-1.0f, -1.0f);
        for (int tile = t_begin; tile < t_end; ++tile) {
            const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile];
            const int count = min(TM, prm.layer_S[layer] - row0);
            const int n_lo = node_lo(tile), n_hi = node_hi(tile);
            const bool shared_tile = drainer && !(n_lo == 0 && n_hi == prm.n_nodes);
            if (failed) {
                // keep the named barriers balanced for the warps that have not given up yet
                if (layer != cur_layer) {
                    asm volatile("bar.sync 1, %0;" ::"n"(NCONV * 32) : "memory");
                    asm volatile("bar.sync 1, %0;" ::"n"(NCONV * 32) : "memory");
                    cur_layer = layer;
                }
                if (shared_tile)
                    for (int i = 0; i < 3; ++i) asm volatile("bar.sync 2, %0;" ::"n"(NDR * 32) : "memory");
                continue;
            }
            if (layer != cur_layer) {
                // Every MMA that read the previous basis has completed: this warp left the last tile
                // through its epilogue, which waited for that tile's accumulator.
                asm volatile("bar.sync 1, %0;" ::"n"(NCONV * 32) : "memory");
                if constexpr (MON) flush_monitor(cur_layer);
                const float *U = prm.Ut + (size_t)layer * KP * d;
                float *Bs = reinterpret_cast<float *>(smem + L.b);
                // element (row r of [U_hi | U_lo], entry t): chunk cc = t / 32, 16-byte piece p = (t % 32) / 4
                // lives at  cc * (2 KP * 128) + (r / 8) * 1024 + (r % 8) * 128 + ((p ^ (r % 8)) * 16) bytes
                constexpr int FILL = (KP * 64 + NCONV * 32 - 1) / (NCONV * 32);   // pieces per thread at d = 256
                float4 uu[FILL];
#pragma unroll
                for (int it = 0; it < FILL; ++it) {   // all loads in flight before the first store
                    const int idx = ctid + it * NCONV * 32;
                    uu[it] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (idx < KP * (d / 4)) uu[it] = __ldg(reinterpret_cast<const float4 *>(U) + idx);
                }
#pragma unroll
                for (int it = 0; it < FILL; ++it) {
                    const int idx = ctid + it * NCONV * 32;
                    if (idx >= KP * (d / 4)) continue;
                    const int jrow = idx / (d / 4), t4 = idx - jrow * (d / 4);
                    const float4 u = uu[it];
                    float4 hi, lo;
                    hi.x = cut_tf32(u.x); hi.y = cut_tf32(u.y); hi.z = cut_tf32(u.z); hi.w = cut_tf32(u.w);
                    lo.x = u.x - hi.x; lo.y = u.y - hi.y; lo.z = u.z - hi.z; lo.w = u.w - hi.w;
                    const int cc = t4 / 8, p = t4 & 7;
                    const int r_hi = jrow, r_lo = KP + jrow;
                    const uint32_t o_hi = cc * (2 * KP * 128) + (r_hi >> 3) * 1024 + (r_hi & 7) * 128 + ((p ^ (r_hi & 7)) << 4);
                    const uint32_t o_lo = cc * (2 * KP * 128) + (r_lo >> 3) * 1024 + (r_lo & 7) * 128 + ((p ^ (r_lo & 7)) << 4);
                    *reinterpret_cast<float4 *>(reinterpret_cast<unsigned char *>(Bs) + o_hi) = hi;
                    *reinterpret_cast<float4 *>(reinterpret_cast<unsigned char *>(Bs) + o_lo) = lo;
                }
                const float div = (float)prm.mean_div;
                for (int t = ctid; t < d; t += NCONV * 32) muN[t] = prm.mu[(size_t)layer * d + t] / div;
                fence_proxy_async();  // the tensor core reads the basis through the async proxy
                asm volatile("bar.sync 1, %0;" ::"n"(NCONV * 32) : "memory");
                if (lane == 0) mbar_arrive(b_ready);
                cur_layer = layer;
            }

            // This thread's row of a stage, as a shared-memory address with the row's swizzle folded in: the row is
            // 128-byte aligned and its 16-byte piece v sits at (v ^ (row % 8)) * 16, so piece v of the row in stage s
            // is at  (stage_s + row * 128 + (row % 8) * 16) ^ (v * 16)  -- one xor with a constant per load.
            const uint32_t myrow_x = smem_u32(stage0) + (uint32_t)(32 * q + lane) * 128 + ((uint32_t)(lane & 7) << 4);
            const int r = 32 * q + lane;
            const int64_t gslice = prm.layer_soff[layer] + row0 + r;   // index of this thread's slice in [S]
            const size_t out_off = (size_t)gslice * KP + col0;
            float acc[COLS];
#pragma unroll
            for (int i = 0; i < COLS; ++i) acc[i] = 0.0f;
            for (int n = n_lo; n <= n_hi && !failed; ++n, ++m) {
                if (n < n_hi && converts) {
                    int cc = cc_next;
                    for (; cc < SUBS; cc += ST) {
                        bool ok = mbar_wait(full + s, s_par, abort_flag);
                        ok = ok && mbar_wait(a_empty + ab, ab_par, abort_flag);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) { failed = true; break; }
                        tc_fence_after();
                        const uint32_t row_x = myrow_x + s * (TM * 128);
                        const float *mch = muN + cc * 32;
                        const uint32_t a_hi = tmem_base + lane_base + A_COL0 + ab * 64;
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            float hi[16], lo[16];
#pragma unroll
                            for (int vv = 0; vv < 4; ++vv) {
                                const int v = half * 4 + vv;
                                const float4 x = lds128(row_x ^ (uint32_t)(v << 4));
                                const float4 mm4 = *reinterpret_cast<const float4 *>(mch + v * 4);
                                // two entries per instruction (packed fp32): x - m as fma(m, -1, x), one rounding, the
                                // very value of the plain subtraction
                                const float2 c01 = __ffma2_rn(make_float2(mm4.x, mm4.y), neg1, make_float2(x.x, x.y));
                                const float2 c23 = __ffma2_rn(make_float2(mm4.z, mm4.w), neg1, make_float2(x.z, x.w));
                                if constexpr (MON) e2 = fmaf(c01.x, c01.x, fmaf(c01.y, c01.y, fmaf(c23.x, c23.x, fmaf(c23.y, c23.y, e2))));
                                // hi = the value cut to TF32's 10 mantissa bits (a bit mask: exact in TF32), lo = the
                                // exact remainder, which the tensor core cuts to TF32 itself
                                const float2 h01 = make_float2(cut_tf32(c01.x), cut_tf32(c01.y));
                                const float2 h23 = make_float2(cut_tf32(c23.x), cut_tf32(c23.y));
                                const float2 l01 = __ffma2_rn(h01, neg1, c01), l23 = __ffma2_rn(h23, neg1, c23);
                                hi[4 * vv + 0] = h01.x; hi[4 * vv + 1] = h01.y; hi[4 * vv + 2] = h23.x; hi[4 * vv + 3] = h23.y;
                                lo[4 * vv + 0] = l01.x; lo[4 * vv + 1] = l01.y; lo[4 * vv + 2] = l23.x; lo[4 * vv + 3] = l23.y;
                            }
                            tmem_st16x2_wait(a_hi + half * 16, hi, a_hi + 32 + half * 16, lo);
                        }
                        // The stage is handed back only here, after the stores above have consumed every value
                        // read from it.  Released right after the loads were issued (their results not yet used),
                        // the arrival overtook loads still in flight and the next TMA load overwrote the rows
                        // they were about to read: the second half of a sub-chunk then held the data of the
                        // stage's next occupant.
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) { mbar_arrive(empty + s); mbar_arrive(a_full + ab); }
                        s += ST; if (s >= NS) { s -= NS; s_par ^= 1; }
                        ab += ST; if (ab >= NABUF) { ab -= NABUF; ab_par ^= 1; }
                    }
                    cc_next = cc - SUBS;
                    if (failed) break;
                    if constexpr (MON) {
                        float e = r < count ? e2 : 0.0f;   // rows past the layer's last slice read as zeros: not data
                        e2 = 0.0f;
#pragma unroll
                        for (int o = 16; o >= 1; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
                        if (lane == 0) atomicAdd(mon_s + n, e);
                    }
                }
                // one node behind the conversion, so that the tensor core is never waited for in steady state
                if (n > n_lo && drainer) {
                    float *sn_base = prm.s_nodes.p[n - 1];
                    if (!drain(m - 1, acc, (sn_base && r < count) ? sn_base + out_off : nullptr, n - 1, gslice, r < count))
                        failed = true;
                }
            }
            --m;  // the loop above ran once more than there are nodes
            if (failed) {
                *abort_flag = 1;
                if (shared_tile)
                    for (int i = 0; i < 3; ++i) asm volatile("bar.sync 2, %0;" ::"n"(NDR * 32) : "memory");
                continue;
            }
            if (!drainer) continue;
            if (!shared_tile) {   // the whole tile was ours
                if (r < count) {
                    float *dst = prm.s_sum + out_off;
#pragma unroll
                    for (int v = 0; v < COLS / 4; ++v)
                        *reinterpret_cast<float4 *>(dst + v * 4) =
                            make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
                }
                continue;
            }
            // A shared tile: park this CTA's piece, take a ticket; the CTA that completes the set adds the
            // pieces in CTA order (a fixed order, whoever comes last) and writes the result.
            const long long b_first = cta_of_unit((long long)tile * prm.n_nodes);
            const long long b_last = cta_of_unit((long long)tile * prm.n_nodes + prm.n_nodes - 1);
            auto piece = [&](long long b) {   // slot 2 b: b's first tile, slot 2 b + 1: its last tile
                const int first_tile_of_b = (int)(unit_start(b) / prm.n_nodes);
                return prm.partial + ((size_t)(2 * b + (tile == first_tile_of_b ? 0 : 1)) * TM + r) * KP + col0;
            };
            {
                float *dst = piece(blockIdx.x);
#pragma unroll
                for (int v = 0; v < COLS / 4; ++v)
                    *reinterpret_cast<float4 *>(dst + v * 4) =
                        make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
            }
            __threadfence();
            asm volatile("bar.sync 2, %0;" ::"n"(NDR * 32) : "memory");
            int *ticket = const_cast<int *>(abort_flag) + 1;
            if (warp == 0 && lane == 0) *ticket = atomicAdd(prm.tile_counter + tile, 1);
            asm volatile("bar.sync 2, %0;" ::"n"(NDR * 32) : "memory");
            if (*reinterpret_cast<volatile int *>(ticket) == (int)(b_last - b_first)) {
                __threadfence();
                if (r < count) {
                    float tot[COLS];
#pragma unroll
                    for (int i = 0; i < COLS; ++i) tot[i] = 0.0f;
                    for (long long b = b_first; b <= b_last; ++b) {
                        const float *src = piece(b);
#pragma unroll
                        for (int v = 0; v < COLS / 4; ++v) {
                            const float4 x = __ldcg(reinterpret_cast<const float4 *>(src) + v);
                            tot[4 * v] += x.x; tot[4 * v + 1] += x.y; tot[4 * v + 2] += x.z; tot[4 * v + 3] += x.w;
                        }
                    }
                    float *dst = prm.s_sum + out_off;
#pragma unroll
                    for (int v = 0; v < COLS / 4; ++v)
                        *reinterpret_cast<float4 *>(dst + v * 4) =
                            make_float4(tot[4 * v], tot[4 * v + 1], tot[4 * v + 2], tot[4 * v + 3]);
                }
                if (warp == 0 && lane == 0) prm.tile_counter[tile] = 0;   // ready for the next launch
            }
            asm volatile("bar.sync 2, %0;" ::"n"(NDR * 32) : "memory");   // the ticket word is reused
        }
        if constexpr (MON) {
            asm volatile("bar.sync 1, %0;" ::"n"(NCONV * 32) : "memory");
            flush_monitor(failed ? -1 : cur_layer);
        }
    }

    if (failed) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(prm.error_word, 1 + warp);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == NCONV + 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

}  // namespace

bool project_sum_tc_supported(int d, int k)
{
    return (k == 16 || k == 32) && d % 64 == 0 && d >= 64 && d <= 256;
}

size_t project_sum_tc_smem_bytes(int d, int k) { return smem_layout(d, k, true).total + 1024; }

size_t project_sum_tc_partial_bytes(int num_sms, int k) { return (size_t)2 * num_sms * TM * k * sizeof(float); }

cudaError_t launch_project_sum_tc(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                                  const LayerTables &lt, const NodePtrs<const float> &g, int n_nodes, int mean_div,
                                  const float *Ut, const float *mu, float *s_sum, int32_t *error_word,
                                  const CUtensorMap *tmaps, int n_layers, const int *slots,
                                  const NodePtrs<float> *s_nodes, float *partial, int32_t *tile_counter,
                                  const int32_t *unit_start, int n_ctas, const TcQuant *quant, double *monitor,
                                  int wait_kcycles, int drop_last_load, int64_t slice_base)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    TcParams prm;
    prm.d = d; prm.n_tiles = tiles.n_tiles; prm.n_nodes = n_nodes; prm.mean_div = mean_div;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.layer_S = lt.S;
    prm.Ut = Ut; prm.mu = mu; prm.s_sum = s_sum; prm.error_word = error_word;
    prm.tmaps = tmaps; prm.n_layers = n_layers;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) prm.slot[n] = n < n_nodes ? slots[n] : 0;
    (void)g;
    if (s_nodes) prm.s_nodes = *s_nodes;
    else for (int n = 0; n < GVQ_MAX_NODES; ++n) prm.s_nodes.p[n] = nullptr;
    prm.partial = partial; prm.tile_counter = tile_counter;
    prm.wait_kcycles = wait_kcycles > 0 ? wait_kcycles : WAIT_KCYCLES_DEFAULT;
    prm.drop_last_load = drop_last_load; prm.slice_base = slice_base;
    (void)num_sms;
    const int grid = n_ctas;
    for (int b = 0; b <= n_ctas; ++b) prm.ustart[b] = unit_start[b];
    const size_t smem = smem_layout(d, k, quant != nullptr).total + 1024;  // slack for the 1024-byte alignment of the base
    prm.levels = quant ? quant->levels : 0;
    prm.seed = quant ? quant->seed : 0;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) {
        prm.q_nodes.p[n] = quant && quant->q_nodes ? quant->q_nodes->p[n] : nullptr;
        prm.norms.p[n] = quant && quant->norms ? quant->norms->p[n] : nullptr;
    }
    auto launch = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(threads_of(quant != nullptr));
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, prm);
    };
    prm.monitor = monitor;
    if (quant) return k == 16 ? launch(project_sum_tc_kernel<16, true, false>) : launch(project_sum_tc_kernel<32, true, false>);
    if (monitor) return k == 16 ? launch(project_sum_tc_kernel<16, false, true>) : launch(project_sum_tc_kernel<32, false, true>);
    return k == 16 ? launch(project_sum_tc_kernel<16, false, false>) : launch(project_sum_tc_kernel<32, false, false>);
}

}  // namespace gvq
