// The exchange buffer of Algorithm 1: what a node sends to its successor for one segment of the gradient,
//   x = [ compressed slices  S x k | uncompressed tail entries  T ]      (floats)
// The compressed part is written by the projection kernels; the kernels here move the tails (layer_len % d
// entries per layer, a few hundred floats in all) between flat gradients and the buffer, and add a received
// buffer to the node's own one (the "adds g'_n to g'" step of the compression round).
#include <algorithm>

#include "gvq_internal.h"
#include "sm100_ptx.cuh"

namespace gvq {
namespace {

struct TailPackParams {
    int n_nodes;
    const int64_t *tail_off;   // [n_tails] offset in a flat gradient
    const int64_t *tail_pos;   // [n_tails] offset in the tail part of an exchange buffer
    const int32_t *tail_len;
    NodePtrs<const float> g;
    float *x_tail;
};

// x_tail[pos + e] = sum over the local nodes of g_n[off + e], node order.
// Both tail kernels are launched BEFORE the projection / decompression they accompany, as links of the same
// chain of programmatic dependent launches: they let their successor start at once (its set-up overlaps this
// handful of blocks; it waits for their completion before it touches memory) and themselves start while their
// predecessor drains, waiting for its completion before their first access.
__global__ void tail_pack_kernel(const __grid_constant__ TailPackParams prm)
{
    ptx::launch_dependents();
    ptx::grid_dependency_wait();
    const int64_t off = prm.tail_off[blockIdx.x], pos = prm.tail_pos[blockIdx.x];
    const int len = prm.tail_len[blockIdx.x];
    for (int e = threadIdx.x; e < len; e += blockDim.x) {
        float acc = prm.g.p[0][off + e];
        for (int n = 1; n < prm.n_nodes; ++n) acc += prm.g.p[n][off + e];
        prm.x_tail[pos + e] = acc;
    }
}

__global__ void tail_unpack_kernel(const int64_t *__restrict__ tail_off, const int64_t *__restrict__ tail_pos,
                                   const int32_t *__restrict__ tail_len, const float *__restrict__ x_tail,
                                   float *__restrict__ g_hat)
{
    ptx::launch_dependents();
    ptx::grid_dependency_wait();
    const int64_t off = tail_off[blockIdx.x], pos = tail_pos[blockIdx.x];
    const int len = tail_len[blockIdx.x];
    for (int e = threadIdx.x; e < len; e += blockDim.x) g_hat[off + e] = x_tail[pos + e];
}

// x_acc += x_in: 12 bytes of traffic per float, no reuse; 128-bit accesses, two per thread in flight
__global__ void __launch_bounds__(256) accumulate_kernel(float *__restrict__ x_acc, const float *__restrict__ x_in,
                                                         int64_t n)
{
    const int64_t n4 = n / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    float4 *a4 = reinterpret_cast<float4 *>(x_acc);
    const float4 *b4 = reinterpret_cast<const float4 *>(x_in);
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + stride < n4; i += 2 * stride) {
        float4 a0 = a4[i], a1 = a4[i + stride];
        const float4 b0 = __ldg(b4 + i), b1 = __ldg(b4 + i + stride);
        a0.x += b0.x; a0.y += b0.y; a0.z += b0.z; a0.w += b0.w;
        a1.x += b1.x; a1.y += b1.y; a1.z += b1.z; a1.w += b1.w;
        a4[i] = a0; a4[i + stride] = a1;
    }
    if (i < n4) {
        float4 a0 = a4[i];
        const float4 b0 = __ldg(b4 + i);
        a0.x += b0.x; a0.y += b0.y; a0.z += b0.z; a0.w += b0.w;
        a4[i] = a0;
    }
    if (blockIdx.x == 0 && threadIdx.x < (int)(n - n4 * 4)) x_acc[n4 * 4 + threadIdx.x] += x_in[n4 * 4 + threadIdx.x];
}

// Per-layer compressed length (Eq. 6 layer by layer): the exchange buffer without the coordinates k_l .. k - 1 of
// every slice of layer l, which a masked basis (gvq_mask_basis) makes exact zeros -- what crosses a link is then
// sum_l S_l k_l + T floats instead of S k + T.  grid (chunks, n_layers + 1): blockIdx.y = layer, the last one the tails.
// PACK: x [S][k] | tails  ->  xp [sum S_l k_l] | tails;  otherwise the inverse (dropped coordinates come back as 0).
template <bool PACK>
__global__ void __launch_bounds__(256) exchange_pack_kernel(int k, int n_layers, const int64_t *__restrict__ layer_soff,
                                                            const int32_t *__restrict__ layer_S,
                                                            const int32_t *__restrict__ layer_k,
                                                            const int64_t *__restrict__ packed_off, int64_t S_total,
                                                            int64_t n_tail, const float *__restrict__ src, float *__restrict__ dst)
{
    const int layer = blockIdx.y;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (layer == n_layers) {   // the tails travel as they are, behind the compressed part
        const int64_t full0 = S_total * k, pack0 = packed_off[n_layers];
        for (int64_t e = t0; e < n_tail; e += stride) dst[(PACK ? pack0 : full0) + e] = src[(PACK ? full0 : pack0) + e];
        return;
    }
    const int kl = layer_k[layer];
    const int64_t S = layer_S[layer], row0 = layer_soff[layer], p0 = packed_off[layer];
    if (PACK) {
        for (int64_t e = t0; e < S * kl; e += stride) {
            const int64_t i = e / kl;
            dst[p0 + e] = src[(row0 + i) * k + (e - i * kl)];
        }
    } else {
        for (int64_t e = t0; e < S * k; e += stride) {
            const int64_t i = e / k;
            const int j = (int)(e - i * k);
            dst[row0 * k + e] = j < kl ? src[p0 + i * kl + j] : 0.0f;
        }
    }
}

template <typename K, typename... Args>
cudaError_t launch_chained(cudaStream_t st, int blocks, K kernel, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(128);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace

cudaError_t launch_tail_pack(cudaStream_t st, const LayerTables &lt, const NodePtrs<const float> &g, int n_nodes,
                             float *x_tail)
{
    if (lt.n_tails == 0) return cudaSuccess;
    TailPackParams prm;
    prm.n_nodes = n_nodes; prm.tail_off = lt.tail_off; prm.tail_pos = lt.tail_pos; prm.tail_len = lt.tail_len;
    prm.g = g; prm.x_tail = x_tail;
    return launch_chained(st, lt.n_tails, tail_pack_kernel, prm);
}

cudaError_t launch_tail_unpack(cudaStream_t st, const LayerTables &lt, const float *x_tail, float *g_hat)
{
    if (lt.n_tails == 0) return cudaSuccess;
    return launch_chained(st, lt.n_tails, tail_unpack_kernel, (const int64_t *)lt.tail_off, (const int64_t *)lt.tail_pos,
                          (const int32_t *)lt.tail_len, x_tail, g_hat);
}

cudaError_t launch_exchange_pack(cudaStream_t st, int num_sms, int k, int n_layers, const LayerTables &lt,
                                 const int32_t *layer_k, const int64_t *packed_off, int64_t S_total, int64_t n_tail,
                                 const float *src, float *dst, bool pack)
{
    const dim3 grid((unsigned)std::max(1, 4 * num_sms / (n_layers + 1)), (unsigned)(n_layers + 1));
    if (pack)
        exchange_pack_kernel<true><<<grid, 256, 0, st>>>(k, n_layers, lt.soff, lt.S, layer_k, packed_off, S_total, n_tail, src, dst);
    else
        exchange_pack_kernel<false><<<grid, 256, 0, st>>>(k, n_layers, lt.soff, lt.S, layer_k, packed_off, S_total, n_tail, src, dst);
    return cudaGetLastError();
}

cudaError_t launch_exchange_accumulate(cudaStream_t st, int num_sms, float *x_acc, const float *x_in, int64_t n)
{
    if (n <= 0) return cudaSuccess;
    const int64_t n4 = n / 4;
    int64_t blocks = (n4 + 2 * 256 - 1) / (2 * 256);
    if (blocks > (int64_t)num_sms * 8) blocks = (int64_t)num_sms * 8;
    if (blocks < 1) blocks = 1;
    accumulate_kernel<<<(unsigned)blocks, 256, 0, st>>>(x_acc, x_in, n);
    return cudaGetLastError();
}

}  // namespace gvq
