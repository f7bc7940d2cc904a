// Projection fused with the N-way compressed-domain sum (Eq. 3 + Eq. 4), FP32-pipe form.
//
//   s_sum[i] = sum_n  Ut_l (x_{n,i} - mu_l / N)          for every slice i of every layer l
//
// One persistent CTA per SM walks a contiguous range of tiles (<= 256 slices of one layer).
// For a tile it streams node after node, 32 columns of the slices at a time, through a
// 3-stage cp.async ring in shared memory; Ut (transposed, padded) and mu / N stay in shared
// memory while the layer does not change.  Each thread owns 4 slices x KT outputs and keeps
// their sums over ALL nodes in registers, so a raw gradient entry is read from HBM exactly
// once and the per-node compressed vectors never leave the chip (unless asked for).
#include "gvq_internal.h"

namespace gvq {
namespace {

constexpr int TS = kProjectRows;  // slices per tile
constexpr int NT = 256;           // threads per CTA
constexpr int RT = 4;             // slices per thread
constexpr int CGT = 4;            // column groups (threads sharing a slice)
constexpr int NSTAGE = 3;

struct ProjectParams {
    int d, k, n_tiles, n_nodes, mean_div;
    const int32_t *tile_layer, *tile_row0;
    const int64_t *layer_off, *layer_soff;
    const int32_t *layer_S;
    const float *Ut, *mu;
    float *s_sum;
    NodePtrs<const float> g;
    NodePtrs<float> s_nodes;
};

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, int src_bytes)
{
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

// KT: outputs per thread and pass; P: passes (k <= 4 * KT * P).
template <int KT, int P, bool PER_NODE>
__global__ void __launch_bounds__(NT, 1) project_sum_kernel(const __grid_constant__ ProjectParams prm)
{
    extern __shared__ __align__(16) float smem[];
    const int d = prm.d, k = prm.k;
    constexpr int KPAD = CGT * KT * P;
    constexpr int KS = KPAD + 4;                 // row stride of the transposed basis
    const int DC = d < 32 ? d : 32;              // columns per pipeline step
    const int XS = DC + 4;                       // row stride of a staged chunk
    const int nchunks = d / DC;
    float *Us = smem;                            // [d][KS]   Us[t][j] = Ut[j][t]
    float *muN = Us + (size_t)d * KS;            // [d]       mu / N
    float *stage = muN + d;                      // [NSTAGE][TS][XS]
    const int stage_floats = TS * XS;

    const int tid = threadIdx.x;
    const int cg = tid & (CGT - 1), rg = tid / CGT;  // rows rg + 64 * i

    const int G = gridDim.x;
    const int t_begin = (int)(((long long)blockIdx.x * prm.n_tiles) / G);
    const int t_end = (int)(((long long)(blockIdx.x + 1) * prm.n_tiles) / G);
    int cur_layer = -1;

    for (int tile = t_begin; tile < t_end; ++tile) {
        const int layer = prm.tile_layer[tile];
        const int row0 = prm.tile_row0[tile];
        const int count = min(TS, prm.layer_S[layer] - row0);
        const int64_t goff = prm.layer_off[layer] + (int64_t)row0 * d;

        if (layer != cur_layer) {
            __syncthreads();  // nobody still reads the old basis
            const float *U = prm.Ut + (size_t)layer * k * d;
            for (int idx = tid; idx < KPAD * d; idx += NT) {
                const int j = idx / d, t = idx - j * d;
                Us[t * KS + j] = (j < k) ? U[(size_t)j * d + t] : 0.0f;
            }
            const float *m = prm.mu + (size_t)layer * d;
            const float div = (float)prm.mean_div;
            for (int t = tid; t < d; t += NT) muN[t] = m[t] / div;
            cur_layer = layer;
            __syncthreads();
        }

        float acc[P][RT][KT];
        float tot[PER_NODE ? P : 1][PER_NODE ? RT : 1][PER_NODE ? KT : 1];
#pragma unroll
        for (int p = 0; p < P; ++p)
#pragma unroll
            for (int i = 0; i < RT; ++i)
#pragma unroll
                for (int c = 0; c < KT; ++c) {
                    acc[p][i][c] = 0.0f;
                    if constexpr (PER_NODE) tot[p][i][c] = 0.0f;
                }

        const int nsteps = prm.n_nodes * nchunks;
        const int units = TS * (DC / 4);  // 16-byte pieces of one chunk
        auto issue = [&](int step) {
            const int n = step / nchunks, ch = step - n * nchunks;
            const float *src = prm.g.p[n] + goff + ch * DC;
            float *dst = stage + (step % NSTAGE) * stage_floats;
            for (int u = tid; u < units; u += NT) {
                const int r = u / (DC / 4), c4 = u - r * (DC / 4);
                const bool valid = r < count;
                cp_async16(dst + r * XS + c4 * 4, valid ? src + (size_t)r * d + c4 * 4 : src, valid ? 16 : 0);
            }
        };
        for (int s = 0; s < NSTAGE - 1; ++s) {
            if (s < nsteps) issue(s);
            cp_async_commit();
        }

        for (int step = 0; step < nsteps; ++step) {
            if (step + NSTAGE - 1 < nsteps) issue(step + NSTAGE - 1);
            cp_async_commit();
            cp_async_wait<NSTAGE - 1>();
            __syncthreads();

            const int n = step / nchunks, ch = step - n * nchunks;
            const float *xs = stage + (step % NSTAGE) * stage_floats;
            const float *us = Us + (size_t)ch * DC * KS + cg * KT;
            const float *ms = muN + ch * DC;
            for (int t4 = 0; t4 < DC / 4; ++t4) {
                const float4 m4 = *reinterpret_cast<const float4 *>(ms + t4 * 4);
                float x[RT][4];
#pragma unroll
                for (int i = 0; i < RT; ++i) {
                    const float4 v = *reinterpret_cast<const float4 *>(xs + (rg + 64 * i) * XS + t4 * 4);
                    x[i][0] = v.x - m4.x; x[i][1] = v.y - m4.y; x[i][2] = v.z - m4.z; x[i][3] = v.w - m4.w;
                }
#pragma unroll
                for (int tt = 0; tt < 4; ++tt) {
#pragma unroll
                    for (int p = 0; p < P; ++p) {
                        float u[KT];
                        const float *up = us + (size_t)(t4 * 4 + tt) * KS + p * (CGT * KT);
                        if constexpr (KT >= 4) {
#pragma unroll
                            for (int c = 0; c < KT; c += 4) {
                                const float4 v = *reinterpret_cast<const float4 *>(up + c);
                                u[c] = v.x; u[c + 1] = v.y; u[c + 2] = v.z; u[c + 3] = v.w;
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < KT; ++c) u[c] = up[c];
                        }
#pragma unroll
                        for (int i = 0; i < RT; ++i)
#pragma unroll
                            for (int c = 0; c < KT; ++c) acc[p][i][c] = fmaf(x[i][tt], u[c], acc[p][i][c]);
                    }
                }
            }

            if constexpr (PER_NODE) if (ch == nchunks - 1) {  // node n is complete: emit s_n, add it to the total
                float *sn = prm.s_nodes.p[n];
#pragma unroll
                for (int p = 0; p < P; ++p)
#pragma unroll
                    for (int i = 0; i < RT; ++i) {
                        const int r = rg + 64 * i;
#pragma unroll
                        for (int c = 0; c < KT; ++c) {
                            const int col = p * (CGT * KT) + cg * KT + c;
                            if (r < count && col < k)
                                sn[(size_t)(prm.layer_soff[layer] + row0 + r) * k + col] = acc[p][i][c];
                            tot[p][i][c] += acc[p][i][c];
                            acc[p][i][c] = 0.0f;
                        }
                    }
            }
            __syncthreads();  // the chunk may be overwritten by the next iteration's copies
        }

#pragma unroll
        for (int p = 0; p < P; ++p)
#pragma unroll
            for (int i = 0; i < RT; ++i) {
                const int r = rg + 64 * i;
#pragma unroll
                for (int c = 0; c < KT; ++c) {
                    const int col = p * (CGT * KT) + cg * KT + c;
                    if (r < count && col < k)
                    {
                        float v;
                        if constexpr (PER_NODE) v = tot[p][i][c]; else v = acc[p][i][c];
                        prm.s_sum[(size_t)(prm.layer_soff[layer] + row0 + r) * k + col] = v;
                    }
                }
            }
    }
}

struct Variant {
    int kt, p;
};
Variant pick_variant(int k)
{
    if (k <= 8) return {2, 1};
    if (k <= 16) return {4, 1};
    if (k <= 32) return {8, 1};
    if (k <= 64) return {8, 2};
    return {8, 4};
}

size_t smem_bytes(int d, int k)
{
    const Variant v = pick_variant(k);
    const int kpad = CGT * v.kt * v.p;
    const int DC = d < 32 ? d : 32;
    return ((size_t)d * (kpad + 4) + d + (size_t)NSTAGE * TS * (DC + 4)) * sizeof(float);
}

template <int KT, int P>
cudaError_t launch_variant(cudaStream_t st, int grid, size_t smem, const ProjectParams &prm, bool per_node)
{
    cudaError_t e;
    if (per_node) {
        e = cudaFuncSetAttribute(project_sum_kernel<KT, P, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        project_sum_kernel<KT, P, true><<<grid, NT, smem, st>>>(prm);
    } else {
        e = cudaFuncSetAttribute(project_sum_kernel<KT, P, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        project_sum_kernel<KT, P, false><<<grid, NT, smem, st>>>(prm);
    }
    return cudaGetLastError();
}

}  // namespace

size_t project_sum_smem_bytes(int d, int k) { return k > 128 ? (size_t)-1 : smem_bytes(d, k); }

cudaError_t launch_project_sum(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                               const LayerTables &lt, const NodePtrs<const float> &g, int n_nodes,
                               int mean_div, const float *Ut, const float *mu, float *s_sum,
                               const NodePtrs<float> *s_nodes)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    ProjectParams prm;
    prm.d = d; prm.k = k; prm.n_tiles = tiles.n_tiles; prm.n_nodes = n_nodes; prm.mean_div = mean_div;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.layer_S = lt.S;
    prm.Ut = Ut; prm.mu = mu; prm.s_sum = s_sum;
    prm.g = g;
    if (s_nodes) prm.s_nodes = *s_nodes;
    else for (int n = 0; n < GVQ_MAX_NODES; ++n) prm.s_nodes.p[n] = nullptr;
    const int grid = tiles.n_tiles < num_sms ? tiles.n_tiles : num_sms;
    const size_t smem = smem_bytes(d, k);
    const Variant v = pick_variant(k);
    const bool pn = s_nodes != nullptr;
    if (v.kt == 2) return launch_variant<2, 1>(st, grid, smem, prm, pn);
    if (v.kt == 4) return launch_variant<4, 1>(st, grid, smem, prm, pn);
    if (v.p == 1) return launch_variant<8, 1>(st, grid, smem, prm, pn);
    if (v.p == 2) return launch_variant<8, 2>(st, grid, smem, prm, pn);
    return launch_variant<8, 4>(st, grid, smem, prm, pn);
}

}  // namespace gvq
