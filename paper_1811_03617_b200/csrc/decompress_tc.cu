// Decompression fused with the mean add (Eq. 5) on the tensor cores (tcgen05, kind::tf32).
//
//   g_hat[i][t] = sum_j Ut_l[j][t] * s_sum[i][j] + mu_l[t]
//
// At k = 32 the FP32 pipe would have to sustain 16 flop per byte written, which it cannot at HBM
// speed; the product is a dense (128 slices x k) x (k x d) contraction per tile, so it runs as
// TF32 MMAs with the same three-product split as the projection (s_hi U_hi + s_hi U_lo + s_lo U_hi,
// hi = value cut to TF32, lo = exact remainder), accumulated in tensor memory.
//
// One persistent CTA per SM walks a contiguous run of (tile, column block) units -- a tile is <= 128
// slices of one layer, a block <= 128 output columns -- the same number of units for every CTA:
//   warps 9-12  per tile: thread <-> slice reads its k compressed values, splits them and stores
//               A_hi / A_lo into tensor memory (four A buffers rotate, up to three tiles ahead);
//               before that they sum the uncompressed tails of the layers (node order, fp32), which
//               would otherwise need a launch of their own
//   warp 8      issues, per block of <= 128 output columns, the 3 k / 8 MMAs (A from tensor memory,
//               U_hi / U_lo of the layer from shared memory, K-major with 128-byte swizzle) into one
//               of two rotating accumulator blocks
//   warps 0-7   epilogue: tcgen05.ld of this warp group's 64 columns of the block, + mu, swizzled store
//               into shared-memory staging tiles, then one tiled TMA store (cp.async.bulk.tensor) per
//               128 slices x 32 entries; the tensor map of the layer drops the rows past its last slice
// The output is written once, by TMA, in full 128-byte rows.  Waits on mbarriers are bounded as in
// the projection kernel.
#include "gvq_internal.h"
#include "sm100_ptx.cuh"

namespace gvq {
namespace {

using namespace ptx;

constexpr int TM = kProjectTcRows;  // slices per tile (MMA M), shares the projection's tile table
constexpr int NEPI = 8;             // epilogue warps: lane quarter q = warp & 3, column group g = warp >> 2
constexpr int NTHREADS = (NEPI + 1 + 4) * 32;   // + MMA issuer + 4 converter warps
constexpr int NABUF = 4;
constexpr uint32_t D_COLS = 128;    // columns of one accumulator block; two blocks: [0, 256)
constexpr uint32_t A_COL0 = 256;    // four A buffers of 64 columns (32 hi + 32 lo): [256, 512)
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t STAGE_BYTES = TM * 128;

struct DtcParams {
    int d, n_tiles;
    const int32_t *tile_layer, *tile_row0;
    const int64_t *layer_soff;
    const int32_t *layer_S;
    const float *s_sum, *Ut, *mu;
    const CUtensorMap *tmaps;  // [layer]: 2-D view (d entries x S_l slices) of g_hat's layer
    int32_t *error_word;
    // the uncompressed tails (layer_len % d entries per layer): g_hat = sum over the nodes, node order
    int n_tails, n_nodes;
    const int64_t *tail_off;
    const int32_t *tail_len;
    float *g_hat;
    NodePtrs<const float> g;
    int32_t ustart[kMaxPartitionCtas + 1];   // CTA b works on units [ustart[b], ustart[b + 1])
    int wait_kcycles;          // limit of every bounded wait, in units of 1024 clocks
    int test_drop;             // test hook: CTA 0's converters do not hand over their first tile, so a wait runs out
};

struct Smem {
    uint32_t bhi, blo, stage, mu, bars, total;
};
__host__ __device__ inline Smem smem_layout(int d)
{
    Smem s;
    s.bhi = 0;                                // [d rows][128 B]  U_hi, row t = entry t, K-major, swizzled
    s.blo = s.bhi + (uint32_t)d * 128;        // [d rows][128 B]  U_lo
    s.stage = s.blo + (uint32_t)d * 128;      // [2 groups][4][128 rows][128 B]  output staging, swizzled
    s.mu = s.stage + 8 * STAGE_BYTES;         // [d] floats
    s.bars = (s.mu + (uint32_t)d * 4 + 15) & ~15u;
    s.total = s.bars + 128;
    return s;
}

template <int KP>
__global__ void __launch_bounds__(NTHREADS, 1) decompress_tc_kernel(const __grid_constant__ DtcParams prm)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int d = prm.d;
    const Smem L = smem_layout(d);
    float *mus = reinterpret_cast<float *>(smem + L.mu);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint64_t *a_full = bars;          // [4] A buffer written       (converters -> MMA)
    uint64_t *a_empty = bars + 4;     // [4] A buffer consumed      (MMA -> converters)
    uint64_t *d_full = bars + 8;      // [2] accumulator complete   (MMA -> epilogue)
    uint64_t *d_empty = bars + 10;    // [2] accumulator read       (epilogue -> MMA)
    uint64_t *b_ready = bars + 12;    // [1] basis of the layer staged
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 13);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x;
    const int n_blocks = (d + 127) / 128;  // output column blocks of <= 128 per tile
    // Work is dealt in units of (tile, column block): a CTA takes a contiguous run, so its first and last tile
    // may be shared with a neighbour, each writing its own column blocks (nothing to combine).  The runs come
    // from the host, balanced by a cost model that charges a run for every layer it touches.
    (void)G;
    const long long u0 = prm.ustart[blockIdx.x], u1 = prm.ustart[blockIdx.x + 1];
    const int t_begin = (int)(u0 / n_blocks);
    const int t_end = u1 > u0 ? (int)((u1 - 1) / n_blocks) + 1 : t_begin;
    auto blk_lo = [&](int tile) { return tile == t_begin ? (int)(u0 - (long long)tile * n_blocks) : 0; };
    auto blk_hi = [&](int tile) { return tile == t_end - 1 ? (int)(u1 - (long long)tile * n_blocks) : n_blocks; };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NABUF; ++i) { mbar_init(a_full + i, 4); mbar_init(a_empty + i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(d_full + i, 1); mbar_init(d_empty + i, NEPI); }
        mbar_init(b_ready, NEPI);
        *abort_flag = 0;
        const_cast<int *>(abort_flag)[2] = prm.wait_kcycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == NEPI) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;
    // The set-up above overlaps the tail of the previous kernel of the stream (normally the projection that
    // produces s_sum); from here on this kernel reads and writes global memory.
    launch_dependents();
    grid_dependency_wait();

    if (warp == NEPI) {
        // ------------------------------------------------------------------ MMA issuer (warp-uniform loop)
        const uint64_t bd0 = make_b_desc(smem_u32(smem + L.bhi));
        const uint32_t bhi_lo = (uint32_t)bd0, bd_hi = (uint32_t)(bd0 >> 32);
        const uint32_t blo_lo = bhi_lo + ((uint32_t)d * 128 >> 4);
        uint32_t ts = 0, bc = 0, layers_seen = 0;
        int cur_layer = -1;
        for (int tile = t_begin; tile < t_end && !failed; ++tile, ++ts) {
            const int layer = prm.tile_layer[tile];
            if (layer != cur_layer) {
                bool ok = mbar_wait(b_ready, layers_seen & 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                ++layers_seen;
                cur_layer = layer;
            }
            const uint32_t ab = ts % NABUF;
            bool ok = mbar_wait(a_full + ab, (ts / NABUF) & 1, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            tc_fence_after();
            const uint32_t a_hi = tmem_base + A_COL0 + ab * 64, a_lo = a_hi + 32;
            const int b_hi = blk_hi(tile);
            for (int blk = blk_lo(tile); blk < b_hi; ++blk, ++bc) {
                const uint32_t hb = bc & 1;
                ok = mbar_wait(d_empty + hb, ((bc >> 1) & 1) ^ 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                tc_fence_after();
                const int nb = min(128, d - blk * 128);
                const uint32_t idesc = make_idesc(nb);
                const uint32_t d_tmem = tmem_base + hb * D_COLS;
                const uint32_t row_off = (uint32_t)blk * (128 * 128 >> 4);  // 128 rows of 128 bytes, in 16-byte units
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < KP / 8; ++kk)
                        tc_mma_tf32_ts(d_tmem, a_hi + kk * 8, bhi_lo + row_off + kk * 2, bd_hi, idesc, kk != 0);
#pragma unroll
                    for (int kk = 0; kk < KP / 8; ++kk)
                        tc_mma_tf32_ts(d_tmem, a_hi + kk * 8, blo_lo + row_off + kk * 2, bd_hi, idesc, 1u);
#pragma unroll
                    for (int kk = 0; kk < KP / 8; ++kk)
                        tc_mma_tf32_ts(d_tmem, a_lo + kk * 8, bhi_lo + row_off + kk * 2, bd_hi, idesc, 1u);
                    tc_commit(d_full + hb);
                    if (blk == b_hi - 1) tc_commit(a_empty + ab);
                }
                __syncwarp();
            }
        }
    } else if (warp > NEPI) {
        // ------------------------------------------------------------------ A conversion
        // thread <-> slice: read its k compressed values, split, store into A buffer (tile number % NABUF)
        const int q = warp & 3;
        const uint32_t lane_base = (uint32_t)(32 * q) << 16;
        const int r = 32 * q + lane;
        uint32_t ts = 0;
        for (int tile = t_begin; tile < t_end && !failed; ++tile, ++ts) {
            const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile];
            const int count = min(TM, prm.layer_S[layer] - row0);
            const uint32_t ab = ts % NABUF;
            const float *src = prm.s_sum + (size_t)(prm.layer_soff[layer] + row0 + r) * KP;
            float4 x[KP / 4];
#pragma unroll
            for (int v = 0; v < KP / 4; ++v) {
                x[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (r < count) x[v] = __ldcs(reinterpret_cast<const float4 *>(src) + v);
            }
            bool ok = mbar_wait(a_empty + ab, ((ts / NABUF) & 1) ^ 1, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            tc_fence_after();
            const uint32_t a_hi = tmem_base + lane_base + A_COL0 + ab * 64;
#pragma unroll
            for (int part = 0; part < KP / 16; ++part) {
                float hi[16], lo[16];
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const float4 xv = x[part * 4 + v];
                    hi[4 * v + 0] = cut_tf32(xv.x); lo[4 * v + 0] = xv.x - hi[4 * v + 0];
                    hi[4 * v + 1] = cut_tf32(xv.y); lo[4 * v + 1] = xv.y - hi[4 * v + 1];
                    hi[4 * v + 2] = cut_tf32(xv.z); lo[4 * v + 2] = xv.z - hi[4 * v + 2];
                    hi[4 * v + 3] = cut_tf32(xv.w); lo[4 * v + 3] = xv.w - hi[4 * v + 3];
                }
                tmem_st16x2_wait(a_hi + part * 16, hi, a_hi + 32 + part * 16, lo);
            }
            tc_fence_before();
            __syncwarp();
            // (test hook: without this hand-over the MMA warp's bounded wait runs out and the kernel gives up)
            if (lane == 0 && !(prm.test_drop && blockIdx.x == 0 && ts == 0)) mbar_arrive(a_full + ab);
        }
        // the tails, dealt round-robin to the CTAs: a handful of entries each, summed in node order
        for (int t = blockIdx.x; t < prm.n_tails; t += gridDim.x) {
            const int64_t off = prm.tail_off[t];
            const int len = prm.tail_len[t];
            for (int e = (warp - NEPI - 1) * 32 + lane; e < len; e += 128) {
                float acc = 0.0f;   // nodes in ascending order, eight independent loads at a time
                for (int n0 = 0; n0 < prm.n_nodes; n0 += 8) {
                    float v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] = n0 + i < prm.n_nodes ? __ldcs(prm.g.p[n0 + i] + off + e) : 0.0f;
                    if (n0 == 0) { acc = v[0]; v[0] = 0.0f; }
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (n0 + i < prm.n_nodes && (n0 + i) > 0) acc += v[i];
                }
                prm.g_hat[off + e] = acc;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3, g = warp >> 2;
        const uint32_t lane_base = (uint32_t)(32 * q) << 16;
        const int r = 32 * q + lane;                    // slice of the tile = tensor-memory lane
        const int sw = lane & 7;
        unsigned char *stage_g = smem + L.stage + (uint32_t)g * 4 * STAGE_BYTES;
        const bool store_issuer = (q == 0 && lane == 0);
        const int bar_id = 2 + g;
        uint32_t bc = 0;

        int cur_layer = -1;
        for (int tile = t_begin; tile < t_end; ++tile) {
            const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile];
            if (layer != cur_layer) {
                // every MMA that read the previous basis is complete: the last tile's epilogue waited for them
                asm volatile("bar.sync 1, %0;" ::"n"(NEPI * 32) : "memory");
                if (!failed) {
                    const float *U = prm.Ut + (size_t)layer * KP * d;
                    // element (entry t, coordinate j) -> row t of 128 bytes, 16-byte piece (j / 4) ^ (t % 8).
                    // A thread owns entry t: it first issues all k loads of its column of Ut (coalesced along
                    // t, all in flight together), then stores k / 4 pieces of 16 bytes.
                    for (int t = threadIdx.x; t < d; t += NEPI * 32) {   // threads 0 .. 255
                        float u[KP];
#pragma unroll
                        for (int j = 0; j < KP; ++j) u[j] = __ldg(U + (size_t)j * d + t);
#pragma unroll
                        for (int p4 = 0; p4 < KP / 4; ++p4) {
                            const float4 hi = make_float4(cut_tf32(u[4 * p4]), cut_tf32(u[4 * p4 + 1]), cut_tf32(u[4 * p4 + 2]),
                                                          cut_tf32(u[4 * p4 + 3]));
                            const float4 lo = make_float4(u[4 * p4] - hi.x, u[4 * p4 + 1] - hi.y, u[4 * p4 + 2] - hi.z,
                                                          u[4 * p4 + 3] - hi.w);
                            const uint32_t off = (uint32_t)(t >> 3) * 1024 + (t & 7) * 128 + ((p4 ^ (t & 7)) << 4);
                            *reinterpret_cast<float4 *>(smem + L.bhi + off) = hi;
                            *reinterpret_cast<float4 *>(smem + L.blo + off) = lo;
                        }
                    }
                    for (int t = threadIdx.x; t < d; t += NEPI * 32) mus[t] = prm.mu[(size_t)layer * d + t];
                    fence_proxy_async();
                }
                asm volatile("bar.sync 1, %0;" ::"n"(NEPI * 32) : "memory");
                if (!failed && lane == 0) mbar_arrive(b_ready);
                cur_layer = layer;
            }
            const CUtensorMap *tm = prm.tmaps + layer;
            const int b_hi = blk_hi(tile);
            for (int blk = blk_lo(tile); blk < b_hi; ++blk, ++bc) {
                const uint32_t hb = bc & 1;
                const int nb = min(128, d - blk * 128);
                const int nsub = nb / 64;                      // 32-column pieces this group writes
                if (!failed) {
                    bool ok = mbar_wait(d_full + hb, (bc >> 1) & 1, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) failed = true;
                    tc_fence_after();
                }
                // this group's nb / 2 columns of the block: all read at once, staged as nsub swizzled tiles
                const int tcol = g * (nb / 2);                 // first column inside the accumulator block
                const int c0 = blk * 128 + tcol;               // first entry
                unsigned char *stg = stage_g + (bc & 1) * 2 * STAGE_BYTES;
                float v[2][32];
                if (!failed) {
                    tmem_ld32_wait(tmem_base + lane_base + hb * D_COLS + tcol, v[0]);
                    if (nsub == 2) tmem_ld32_wait(tmem_base + lane_base + hb * D_COLS + tcol + 32, v[1]);
                    tc_fence_before();                         // this warp is done with the accumulator block
                    __syncwarp();
                    if (lane == 0) mbar_arrive(d_empty + hb);
                }
                // the TMA stores that last read these staging tiles (two blocks ago) must have finished reading
                if (store_issuer) bulk_wait_group_read<1>();
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                if (!failed) {
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub) {
                        if (sub < nsub) {
                            unsigned char *row = stg + sub * STAGE_BYTES + (size_t)r * 128;
#pragma unroll
                            for (int x = 0; x < 8; ++x) {
                                const float4 m4 = *reinterpret_cast<const float4 *>(mus + c0 + sub * 32 + x * 4);
                                *reinterpret_cast<float4 *>(row + ((x ^ sw) << 4)) =
                                    make_float4(v[sub][4 * x] + m4.x, v[sub][4 * x + 1] + m4.y, v[sub][4 * x + 2] + m4.z,
                                                v[sub][4 * x + 3] + m4.w);
                            }
                        }
                    }
                    fence_proxy_async();  // the TMA stores read the tiles through the async proxy
                }
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                if (store_issuer && !failed) {
                    tma_store_2d(tm, c0, row0, stg);
                    if (nsub == 2) tma_store_2d(tm, c0 + 32, row0, stg + STAGE_BYTES);
                    bulk_commit_group();                       // one group per block
                }
            }
        }
        if (store_issuer) bulk_wait_group_all();
    }

    if (failed) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(prm.error_word, 100 + warp);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == NEPI)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

}  // namespace

cudaError_t launch_decompress_tc(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                                 const LayerTables &lt, const float *s_sum, const float *Ut, const float *mu,
                                 const CUtensorMap *tmaps_of_g_hat, int32_t *error_word,
                                 const NodePtrs<const float> *g_for_tails, int n_nodes, const int32_t *unit_start,
                                 int n_ctas, float *g_hat, int wait_kcycles, int test_drop)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    DtcParams prm;
    prm.n_tails = g_for_tails ? lt.n_tails : 0; prm.n_nodes = n_nodes;
    prm.tail_off = lt.tail_off; prm.tail_len = lt.tail_len; prm.g_hat = g_hat;
    if (g_for_tails) prm.g = *g_for_tails;
    else for (int n = 0; n < GVQ_MAX_NODES; ++n) prm.g.p[n] = nullptr;
    prm.d = d; prm.n_tiles = tiles.n_tiles;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0;
    prm.layer_soff = lt.soff; prm.layer_S = lt.S;
    prm.s_sum = s_sum; prm.Ut = Ut; prm.mu = mu; prm.tmaps = tmaps_of_g_hat; prm.error_word = error_word;
    prm.wait_kcycles = wait_kcycles > 0 ? wait_kcycles : WAIT_KCYCLES_DEFAULT;
    prm.test_drop = test_drop;
    (void)num_sms;
    const int grid = n_ctas;
    for (int b = 0; b <= n_ctas; ++b) prm.ustart[b] = unit_start[b];
    const size_t smem = smem_layout(d).total + 1024;
    auto launch = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(NTHREADS);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, prm);
    };
    return k == 16 ? launch(decompress_tc_kernel<16>) : launch(decompress_tc_kernel<32>);
}

}  // namespace gvq
