// Decompression fused with the mean add (Eq. 5), and the uncompressed tails.
//
//   g_hat[i][t] = sum_j Ut_l[j][t] * s_sum[i][j] + mu_l[t]
//
// One persistent CTA per SM walks a contiguous range of tiles (<= 64 slices of one layer).
// Ut_l (k x d, padded to a multiple of 4 rows) and mu_l stay in shared memory while the layer
// does not change; the tile's compressed vectors are staged in shared memory; each thread
// produces 8 slices x 4 adjacent entries and writes them as 128-bit coalesced stores.  The
// output is written exactly once and nothing but s_sum (k / d of its size) is read.
#include "gvq_internal.h"

namespace gvq {
namespace {

constexpr int TSD = kDecompressRows;
constexpr int NT = 256;
constexpr int RT = 8;

struct DecompressParams {
    int d, k, n_tiles;
    const int32_t *tile_layer, *tile_row0;
    const int64_t *layer_off, *layer_soff;
    const int32_t *layer_S;
    const float *s_sum, *Ut, *mu;
    float *g_hat;
};

__global__ void __launch_bounds__(NT, 2) decompress_kernel(const __grid_constant__ DecompressParams prm)
{
    extern __shared__ __align__(16) float smem[];
    const int d = prm.d, k = prm.k;
    const int k4 = (k + 3) & ~3;
    float *Us = smem;                    // [k4][d]
    float *ms = Us + (size_t)k4 * d;     // [d]
    float *ss = ms + d;                  // [TSD][k4]
    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int t_begin = (int)(((long long)blockIdx.x * prm.n_tiles) / G);
    const int t_end = (int)(((long long)(blockIdx.x + 1) * prm.n_tiles) / G);
    const int d4 = d / 4;
    const int items = (TSD / RT) * d4;
    int cur_layer = -1;

    for (int tile = t_begin; tile < t_end; ++tile) {
        const int layer = prm.tile_layer[tile];
        const int row0 = prm.tile_row0[tile];
        const int count = min(TSD, prm.layer_S[layer] - row0);
        __syncthreads();  // previous tile's readers are done with ss (and Us)
        if (layer != cur_layer) {
            const float *U = prm.Ut + (size_t)layer * k * d;
            for (int idx = tid; idx < k4 * d4; idx += NT) {
                const int j = idx / d4, c4 = idx - j * d4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < k) v = *reinterpret_cast<const float4 *>(U + (size_t)j * d + c4 * 4);
                *reinterpret_cast<float4 *>(Us + (size_t)j * d + c4 * 4) = v;
            }
            for (int t = tid; t < d; t += NT) ms[t] = prm.mu[(size_t)layer * d + t];
            cur_layer = layer;
        }
        const float *src = prm.s_sum + (size_t)(prm.layer_soff[layer] + row0) * k;
        for (int idx = tid; idx < TSD * k4; idx += NT) {
            const int r = idx / k4, j = idx - r * k4;
            ss[idx] = (r < count && j < k) ? src[(size_t)r * k + j] : 0.0f;
        }
        __syncthreads();

        float *out = prm.g_hat + prm.layer_off[layer] + (int64_t)row0 * d;
        for (int it = tid; it < items; it += NT) {
            const int rb = it / d4, c4 = it - rb * d4;
            const float4 m4 = *reinterpret_cast<const float4 *>(ms + c4 * 4);
            float acc[RT][4];
#pragma unroll
            for (int r = 0; r < RT; ++r) { acc[r][0] = m4.x; acc[r][1] = m4.y; acc[r][2] = m4.z; acc[r][3] = m4.w; }
            for (int j = 0; j < k4; j += 4) {
                float4 u[4];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    u[jj] = *reinterpret_cast<const float4 *>(Us + (size_t)(j + jj) * d + c4 * 4);
#pragma unroll
                for (int r = 0; r < RT; ++r) {
                    const float4 s4 = *reinterpret_cast<const float4 *>(ss + (rb * RT + r) * k4 + j);
                    const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        acc[r][0] = fmaf(u[jj].x, sv[jj], acc[r][0]);
                        acc[r][1] = fmaf(u[jj].y, sv[jj], acc[r][1]);
                        acc[r][2] = fmaf(u[jj].z, sv[jj], acc[r][2]);
                        acc[r][3] = fmaf(u[jj].w, sv[jj], acc[r][3]);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                const int row = rb * RT + r;
                if (row < count)
                    __stcs(reinterpret_cast<float4 *>(out + (size_t)row * d + c4 * 4),
                           make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]));
            }
        }
    }
}

struct TailParams {
    int n_nodes;
    const int64_t *tail_off;
    const int32_t *tail_len;
    NodePtrs<const float> g;
    float *g_hat;
};

// One CTA per layer with a tail: g_hat[e] = g_0[e] + g_1[e] + ... in node order.
__global__ void tail_sum_kernel(const __grid_constant__ TailParams prm)
{
    const int64_t off = prm.tail_off[blockIdx.x];
    const int len = prm.tail_len[blockIdx.x];
    for (int e = threadIdx.x; e < len; e += blockDim.x) {
        float acc = prm.g.p[0][off + e];
        for (int n = 1; n < prm.n_nodes; ++n) acc += prm.g.p[n][off + e];
        prm.g_hat[off + e] = acc;
    }
}

}  // namespace

size_t decompress_smem_bytes(int d, int k)
{
    const int k4 = (k + 3) & ~3;
    return ((size_t)k4 * d + d + (size_t)TSD * k4) * sizeof(float);
}

cudaError_t launch_decompress(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                              const LayerTables &lt, const float *s_sum, const float *Ut, const float *mu,
                              float *g_hat)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    DecompressParams prm;
    prm.d = d; prm.k = k; prm.n_tiles = tiles.n_tiles;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.layer_S = lt.S;
    prm.s_sum = s_sum; prm.Ut = Ut; prm.mu = mu; prm.g_hat = g_hat;
    const size_t smem = decompress_smem_bytes(d, k);
    cudaError_t e = cudaFuncSetAttribute(decompress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int per_sm = smem * 2 <= 220 * 1024 ? 2 : 1;
    int grid = num_sms * per_sm;
    if (grid > tiles.n_tiles) grid = tiles.n_tiles;
    decompress_kernel<<<grid, NT, smem, st>>>(prm);
    return cudaGetLastError();
}

cudaError_t launch_tail_sum(cudaStream_t st, const LayerTables &lt, int d, const NodePtrs<const float> &g,
                            int n_nodes, float *g_hat)
{
    (void)d;
    if (lt.n_tails == 0) return cudaSuccess;
    TailParams prm;
    prm.n_nodes = n_nodes; prm.tail_off = lt.tail_off; prm.tail_len = lt.tail_len; prm.g = g; prm.g_hat = g_hat;
    tail_sum_kernel<<<lt.n_tails, 128, 0, st>>>(prm);
    return cudaGetLastError();
}

}  // namespace gvq
