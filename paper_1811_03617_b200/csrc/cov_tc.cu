// Covariance partial sums of the basis fit (Section 2, PCA paragraph) on the 5th-generation tensor cores.
//
//   partial[tile][a][b] = sum over the tile's samples x (all L stored gradients) of (x_a - m_a)(x_b - m_b)
//
// m need only be near the mean: the kernel also returns sum (x - m) per entry, from which the caller gets the
// exact mean and the correction  C = S2 / n - delta delta^T  (delta = mean - m), so the history is read once
// instead of once for the mean and once for the covariance.
//
// A sample is one slice (d entries); a tile holds <= 512 slices of one layer in every stored gradient.
// The work unit is (tile, pair of 128-entry blocks bi <= bj): D[128 x 128] += A B^T with the samples as
// the contraction, A = centred entries of block bi (tensor memory, lane = entry, columns = samples),
// B = centred entries of block bj (shared memory, row = entry, 128 bytes = 32 samples, the K-major
// 128-byte-swizzled layout).  As in the projection every product is three TF32 products,
//      a b ~= a_hi b_hi + a_hi b_lo + a_lo b_hi,
// the first into one accumulator, the two small ones into a second.  The tensor core's accumulator
// rounds toward zero, so the first accumulator is read back and added into registers (round to
// nearest) every 16 chunks of 32 samples; the second carries terms 2^-11 of the first and is read once
// per unit.
//
// One persistent CTA per SM, warp-specialised:
//   producer    one thread: per chunk of 32 samples one 3-D tiled TMA load (entries x slices x stored
//               gradient; box 32 x 32 x 1, 128-byte swizzle, zero fill outside) per 32-entry sub-block
//   warps 0-11  converters, three groups that take the chunks in turn: warp q of a group owns sub-block q of the
//               block(s): lane = entry, reads its entry's 32 samples (one 4-byte load per sample row,
//               conflict-free), subtracts the mean, zeroes samples past the tile's end, splits hi / lo,
//               stores its A row into tensor memory and its B row into shared memory.  The same warps
//               read the accumulators back (group = 48, 48 and 32 of the 128 columns) and write the unit's block.
//   warp 12     the producer (above); warps 13, 14  MMA issuers: a_hi b_hi products / the two cross products, warp-uniform loops with one
//               elected lane issuing
// Every mbarrier wait is bounded; on expiry the CTA records an error word, lets its copies land, frees
// its tensor memory and returns.
#include "gvq_internal.h"
#include "sm100_ptx.cuh"

namespace gvq {
namespace {

using namespace ptx;

constexpr int KC = 32;       // samples per chunk (= one 128-byte row of B)
constexpr int NSLOT = 8;     // raw 16 KB pieces in flight (a chunk of block bi, or of block bj when bi != bj): the loads' latency, not their rate, would bound the kernel with fewer
constexpr int NOP = 3;       // operand buffers: A (hi | lo, 64 columns) in tensor memory, B (hi, lo: 32 KB) in shared
constexpr int PERIOD = 16;   // chunks between read-backs of the main accumulator
constexpr int NG = 3;        // converter groups of four warps; chunk c goes to group c % NG
constexpr int NCW = 4 * NG;  // converter warps
constexpr int NTHREADS = (NCW + 3) * 32;
constexpr uint32_t ACC1 = 0, ACC2 = 128, A_COL0 = 256, TMEM_COLS = 512;
constexpr uint32_t SLOT_BYTES = 16 * 1024, OP_BYTES = 32 * 1024;

struct CovParams {
    int d, L, n_units, n_pairs, nb;
    const int32_t *tile_layer, *tile_row0, *layer_S;
    const float *mean;          // [layers][d]
    const CUtensorMap *maps;    // [layers]: 3-D view (d entries, S_l slices, L stored gradients) of the history
    const int32_t *order;       // [n_units] unit ids, longest first
    float *partial;             // [tiles][d][d]
    double *shift_sum;          // [layers][d]: sum over all samples of (x - mean); `mean` may be approximate
    int32_t *error_word;
    int wait_kcycles;           // limit of every bounded wait, in units of 1024 clocks
    int test_drop;              // test hook: CTA 0's producer leaves out its first load, so a wait runs out
};

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *tmap, int x, int y, int z, uint64_t *bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(NTHREADS, 1) cov_tc_kernel(const __grid_constant__ CovParams prm)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char *slots = smem;                               // [NSLOT][16 KB]
    unsigned char *ops = smem + NSLOT * SLOT_BYTES;            // [NOP][B_hi 16 KB | B_lo 16 KB]
    uint64_t *bars = reinterpret_cast<uint64_t *>(ops + NOP * OP_BYTES);
    uint64_t *full = bars;                // [NSLOT] raw chunk landed            (producer -> converters)
    uint64_t *empty = full + NSLOT;       // [NSLOT] raw chunk consumed          (converters -> producer)
    uint64_t *op_full = empty + NSLOT;    // [NOP]   operands written            (converters -> MMA)
    uint64_t *op_empty = op_full + NOP;   // [NOP]   operands consumed           (MMA -> converters)
    uint64_t *d_full = op_empty + NOP;    // main accumulator complete for a period   (MMA -> read-back)
    uint64_t *d_empty = d_full + 1;       // main accumulator read                     (read-back -> MMA)
    uint64_t *x_full = d_empty + 1;       // cross-term accumulator complete for a unit
    uint64_t *x_empty = x_full + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(x_empty + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d = prm.d;
    if (threadIdx.x == 0) {
        for (int i = 0; i < NSLOT; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 4); }
        for (int i = 0; i < NOP; ++i) { mbar_init(op_full + i, 4); mbar_init(op_empty + i, 2); }
        mbar_init(d_full, 1); mbar_init(d_empty, NCW);
        mbar_init(x_full, 1); mbar_init(x_empty, NCW);
        *abort_flag = 0;
        const_cast<int *>(abort_flag)[2] = prm.wait_kcycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == NCW + 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;

    // Units are dealt from the list sorted longest first, alternately forwards and backwards over the CTAs
    // (CTA b takes entries b, 2G - 1 - b, 2G + b, ...), which evens out the totals.  -1: no unit in this round.
    const int G = gridDim.x;
    const int n_rounds = (prm.n_units + G - 1) / G;
    auto unit_in_round = [&](int i) {
        const int idx = i * G + ((i & 1) ? G - 1 - (int)blockIdx.x : (int)blockIdx.x);
        return idx < prm.n_units ? (int)prm.order[idx] : -1;
    };
    // the geometry of unit u, the same for every role
    struct Unit { int tile, layer, row0, count, bi, bj, cph, n_chunks; };
    auto unit_of = [&](int u) {
        Unit g;
        g.tile = u / prm.n_pairs;
        int pi = u - g.tile * prm.n_pairs;
        g.bi = 0;
        while (pi >= prm.nb - g.bi) { pi -= prm.nb - g.bi; ++g.bi; }
        g.bj = g.bi + pi;
        g.layer = prm.tile_layer[g.tile];
        g.row0 = prm.tile_row0[g.tile];
        g.count = min(kFitRows, prm.layer_S[g.layer] - g.row0);
        g.cph = (g.count + KC - 1) / KC;     // chunks per stored gradient
        g.n_chunks = prm.L * g.cph;
        return g;
    };

    if (warp == NCW) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t sc = 0;   // raw pieces issued so far
            for (int i = 0; i < n_rounds && !failed; ++i) {
                const int u = unit_in_round(i);
                if (u < 0) continue;
                const Unit g = unit_of(u);
                const CUtensorMap *tm = prm.maps + g.layer;
                const int sides = g.bi == g.bj ? 1 : 2;
                for (int ci = 0; ci < g.n_chunks && !failed; ++ci) {
                    const int h = ci / g.cph, cs = ci - h * g.cph;
                    for (int side = 0; side < sides; ++side, ++sc) {
                        const uint32_t s = sc % NSLOT;
                        if (!mbar_wait(empty + s, ((sc / NSLOT) & 1) ^ 1, abort_flag)) { failed = true; break; }
                        if (prm.test_drop && blockIdx.x == 0 && sc == 0) continue;   // test hook: this piece never arrives
                        mbar_arrive_expect_tx(full + s, SLOT_BYTES);
                        unsigned char *dst = slots + (size_t)s * SLOT_BYTES;
                        const int blk = side == 0 ? g.bi : g.bj;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            tma_load_3d(dst + q * 4096, tm, 128 * blk + 32 * q, g.row0 + KC * cs, h, full + s);
                    }
                }
            }
            const uint32_t c = sc;
            if (failed) {   // give the copies already in flight a bounded chance to land before the CTA exits
                for (uint32_t i = c > NSLOT ? c - NSLOT : 0; i < c; ++i)
                    for (int it = 0; it < 100000 && !mbar_try_wait(full + i % NSLOT, (i / NSLOT) & 1); ++it) {}
            }
        }
        failed = __shfl_sync(0xffffffffu, failed, 0);
    } else if (warp > NCW) {
        // ------------------------------------------------------------------ MMA issuers
        const int which = warp - (NCW + 1);   // 0: a_hi b_hi -> ACC1;  1: a_hi b_lo + a_lo b_hi -> ACC2
        const uint32_t idesc = make_idesc(128);
        const uint64_t bd0 = make_b_desc(smem_u32(ops));
        const uint32_t bd0_lo = (uint32_t)bd0, bd0_hi = (uint32_t)(bd0 >> 32);
        uint32_t c = 0, periods = 0, units = 0;
        for (int i = 0; i < n_rounds && !failed; ++i) {
            const int u = unit_in_round(i);
            if (u < 0) continue;
            const Unit g = unit_of(u);
            for (int ci = 0; ci < g.n_chunks; ++ci, ++c) {
                const uint32_t ob = c % NOP;
                bool ok = mbar_wait(op_full + ob, (c / NOP) & 1, abort_flag);
                bool fresh = false;   // the first MMA of a period / unit overwrites its accumulator
                if (which == 0 && ci % PERIOD == 0) {
                    ok = ok && mbar_wait(d_empty, (periods & 1) ^ 1, abort_flag);
                    fresh = true;
                }
                if (which == 1 && ci == 0) {
                    ok = ok && mbar_wait(x_empty, (units & 1) ^ 1, abort_flag);
                    fresh = true;
                }
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                tc_fence_after();
                const uint32_t a_hi = tmem_base + A_COL0 + ob * 64, a_lo = a_hi + 32;
                const uint32_t b_hi = bd0_lo + ob * (OP_BYTES / 16), b_lo = b_hi + 16384 / 16;   // 16-byte units
                if (elect_one()) {
                    if (which == 0) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            tc_mma_tf32_ts(tmem_base + ACC1, a_hi + kk * 8, b_hi + kk * 2, bd0_hi, idesc,
                                           (fresh && kk == 0) ? 0u : 1u);
                    } else {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            tc_mma_tf32_ts(tmem_base + ACC2, a_hi + kk * 8, b_lo + kk * 2, bd0_hi, idesc,
                                           (fresh && kk == 0) ? 0u : 1u);
                        // On a diagonal unit A and B hold the same entries, so a_lo b_hi^T is the transpose of
                        // a_hi b_lo^T: it is not computed; the read-back doubles this accumulator instead and the
                        // reduction symmetrises the block, (X + X^T) / 2 with X = hh + 2 hl.
                        if (g.bi != g.bj) {
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                tc_mma_tf32_ts(tmem_base + ACC2, a_lo + kk * 8, b_hi + kk * 2, bd0_hi, idesc, 1u);
                        }
                    }
                    tc_commit(op_empty + ob);
                    if (which == 0 && (ci % PERIOD == PERIOD - 1 || ci == g.n_chunks - 1)) tc_commit(d_full);
                    if (which == 1 && ci == g.n_chunks - 1) tc_commit(x_full);
                }
                __syncwarp();
                if (which == 0 && (ci % PERIOD == PERIOD - 1 || ci == g.n_chunks - 1)) ++periods;
            }
            ++units;
        }
    } else {
        // ------------------------------------------------------------------ converters + read-back
        const int q = warp & 3, grp = warp >> 2;      // lane quarter = sub-block; group = chunk turn = column range
        const int colg = 48 * grp, nc16 = grp < 2 ? 3 : 2;   // this group's accumulator columns: 16-column pieces
        const uint32_t lane_base = (uint32_t)(32 * q) << 16;
        const int r = 32 * q + lane;                  // this thread's row of A and of B
        uint32_t c = 0, periods = 0, units = 0, sc_base = 0;   // sc_base: raw pieces of the units before this one
        for (int i = 0; i < n_rounds; ++i) {
            const int u = unit_in_round(i);
            if (u < 0) continue;
            const Unit g = unit_of(u);
            const int sides = g.bi == g.bj ? 1 : 2;
            const int ea = 128 * g.bi + r, eb = 128 * g.bj + r;
            const float ma = ea < d ? prm.mean[(size_t)g.layer * d + ea] : 0.0f;
            const float mb = eb < d ? prm.mean[(size_t)g.layer * d + eb] : 0.0f;
            const int n_periods = (g.n_chunks + PERIOD - 1) / PERIOD;
            int drained = 0;
            float s1 = 0.0f;   // this thread's share of the sum of the centred samples of entry ea (diagonal units)
            float sum[48];
#pragma unroll
            for (int i = 0; i < 48; ++i) sum[i] = 0.0f;
            // adds the main accumulator's columns [colg, colg + 16 nc16) of row r into sum and hands it back
            auto read_back = [&]() -> bool {
                bool ok = mbar_wait(d_full, periods & 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) return false;
                tc_fence_after();
                const uint32_t t = tmem_base + lane_base + ACC1 + colg;
#pragma unroll
                for (int pc = 0; pc < 3; ++pc) {
                    if (pc < nc16) {
                        float v[16];
                        tmem_ld16_wait(t + 16 * pc, v);
#pragma unroll
                        for (int i = 0; i < 16; ++i) sum[16 * pc + i] += v[i];
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d_empty);
                ++periods;
                ++drained;
                return true;
            };
            for (int ci = 0; ci < g.n_chunks && !failed; ++ci, ++c) {
                if ((int)(c % NG) != grp) continue;   // another group's chunk
                // a finished period is read back two chunks late, when the tensor core has long left it
                while (!failed && drained < n_periods && (drained + 1) * PERIOD + 2 <= ci)
                    if (!read_back()) failed = true;
                if (failed) break;
                const uint32_t ob = c % NOP;
                const uint32_t sc = sc_base + (uint32_t)ci * sides, s = sc % NSLOT, s2 = (sc + 1) % NSLOT;
                bool ok = mbar_wait(full + s, (sc / NSLOT) & 1, abort_flag);
                if (sides == 2) ok = ok && mbar_wait(full + s2, ((sc + 1) / NSLOT) & 1, abort_flag);
                ok = ok && mbar_wait(op_empty + ob, ((c / NOP) & 1) ^ 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                tc_fence_after();
                const int h = ci / g.cph, cs = ci - h * g.cph;
                const int nvalid = min(KC, g.count - KC * cs);   // samples of this chunk inside the tile
                const unsigned char *raw[2] = {slots + (size_t)s * SLOT_BYTES + q * 4096 + (lane & 3) * 4,
                                               slots + (size_t)s2 * SLOT_BYTES + q * 4096 + (lane & 3) * 4};
                unsigned char *bop = ops + (size_t)ob * OP_BYTES + (r >> 3) * 1024 + (r & 7) * 128;
                const uint32_t a_t = tmem_base + lane_base + A_COL0 + ob * 64;
#pragma unroll
                for (int side = 0; side < 2; ++side) {   // 0: block bi -> A (and B when bi == bj); 1: block bj -> B
                    if (side == 1 && g.bi == g.bj) break;
                    const float m = side == 0 ? ma : mb;
                    const unsigned char *src = raw[side];
#pragma unroll
                    for (int part = 0; part < 2; ++part) {   // 16 samples at a time keeps the register count down
                        float hi[16], lo[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int smp = 16 * part + i;
                            const float x = *reinterpret_cast<const float *>(src + smp * 128 + (((lane >> 2) ^ (smp & 7)) << 4));
                            const float v = smp < nvalid ? x - m : 0.0f;
                            hi[i] = cut_tf32(v);
                            lo[i] = v - hi[i];
                            if (side == 0) s1 += v;
                        }
                        if (side == 0) tmem_st16x2_wait(a_t + 16 * part, hi, a_t + 32 + 16 * part, lo);
                        if (side == 1 || g.bi == g.bj) {
#pragma unroll
                            for (int pp = 0; pp < 4; ++pp) {
                                const int p = 4 * part + pp;
                                const uint32_t off = (uint32_t)((p ^ (r & 7)) << 4);
                                *reinterpret_cast<float4 *>(bop + off) = make_float4(hi[4 * pp], hi[4 * pp + 1], hi[4 * pp + 2], hi[4 * pp + 3]);
                                *reinterpret_cast<float4 *>(bop + 16384 + off) = make_float4(lo[4 * pp], lo[4 * pp + 1], lo[4 * pp + 2], lo[4 * pp + 3]);
                            }
                        }
                    }
                }
                // the raw chunk goes back only now that every value read from it has been used
                fence_proxy_async();   // the tensor core reads B through the async proxy
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(empty + s);
                    if (sides == 2) mbar_arrive(empty + s2);
                    mbar_arrive(op_full + ob);
                }
            }
            sc_base += (uint32_t)g.n_chunks * sides;
            if (!failed) {
                while (drained < n_periods)
                    if (!read_back()) { failed = true; break; }
            }
            if (failed) { *abort_flag = 1; continue; }
            // the cross terms, once per unit
            {
                bool ok = mbar_wait(x_full, units & 1, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; *abort_flag = 1; continue; }
                tc_fence_after();
                const uint32_t t = tmem_base + lane_base + ACC2 + colg;
#pragma unroll
                for (int pc = 0; pc < 3; ++pc) {
                    if (pc < nc16) {
                        float v[16];
                        tmem_ld16_wait(t + 16 * pc, v);
                        const float w2 = g.bi == g.bj ? 2.0f : 1.0f;
#pragma unroll
                        for (int i = 0; i < 16; ++i) sum[16 * pc + i] = fmaf(w2, v[i], sum[16 * pc + i]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(x_empty);
            }
            if (g.bi == g.bj && ea < d) atomicAdd(prm.shift_sum + (size_t)g.layer * d + ea, (double)s1);
            const int col0 = 128 * g.bj + colg;
            if (ea < d) {
                float *dst = prm.partial + ((size_t)g.tile * d + ea) * d + col0;
#pragma unroll
                for (int pc = 0; pc < 3; ++pc) {
                    if (pc < nc16 && col0 + 16 * pc < d) {   // d is a multiple of 64: a 16-column piece is in or out
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4)
                            *reinterpret_cast<float4 *>(dst + 16 * pc + 4 * v4) =
                                make_float4(sum[16 * pc + 4 * v4], sum[16 * pc + 4 * v4 + 1], sum[16 * pc + 4 * v4 + 2],
                                            sum[16 * pc + 4 * v4 + 3]);
                    }
                }
            }
            ++units;
        }
    }

    if (failed) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(prm.error_word, 100 + warp);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == NCW + 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

}  // namespace

bool cov_tc_supported(int d) { return d % 64 == 0 && d >= 64 && d <= 256; }

cudaError_t launch_cov_tc(cudaStream_t st, int num_sms, int d, int L, const TileTable &tiles, const LayerTables &lt,
                          const float *mean, const CUtensorMap *maps, const int32_t *unit_order, float *partial,
                          double *shift_sum, int32_t *error_word, int wait_kcycles, int test_drop)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    CovParams prm;
    prm.d = d; prm.L = L;
    prm.nb = (d + 127) / 128;
    prm.n_pairs = prm.nb * (prm.nb + 1) / 2;
    prm.n_units = tiles.n_tiles * prm.n_pairs;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0; prm.layer_S = lt.S;
    prm.mean = mean; prm.maps = maps; prm.order = unit_order; prm.partial = partial; prm.shift_sum = shift_sum; prm.error_word = error_word;
    prm.wait_kcycles = wait_kcycles > 0 ? wait_kcycles : ptx::WAIT_KCYCLES_DEFAULT;
    prm.test_drop = test_drop;
    const size_t smem = (size_t)NSLOT * SLOT_BYTES + (size_t)NOP * OP_BYTES + 256 + 1024;
    cudaError_t e = cudaFuncSetAttribute(cov_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int grid = prm.n_units < num_sms ? prm.n_units : num_sms;
    cov_tc_kernel<<<grid, NTHREADS, smem, st>>>(prm);
    return cudaGetLastError();
}

}  // namespace gvq
