// Compressed-domain aggregation on materialised buffers (Eq. 4) and the stochastic scalar
// quantizer of compressed vectors with its dequantise-and-sum counterpart.
#include "gvq_internal.h"

namespace gvq {
namespace {

struct AggParams {
    int n_nodes;
    int64_t count;
    NodePtrs<const float> s;
    float *out;
};

// out[e] = s_0[e] + s_1[e] + ... (node order), 128-bit accesses, grid-stride.
__global__ void __launch_bounds__(256) aggregate_kernel(const __grid_constant__ AggParams prm)
{
    const int64_t n4 = prm.count / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += stride) {
        float4 acc = __ldcs(reinterpret_cast<const float4 *>(prm.s.p[0]) + e);
        for (int n = 1; n < prm.n_nodes; ++n) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(prm.s.p[n]) + e);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        reinterpret_cast<float4 *>(prm.out)[e] = acc;
    }
    // up to three trailing entries
    if (blockIdx.x == 0 && threadIdx.x < (int)(prm.count - n4 * 4)) {
        const int64_t e = n4 * 4 + threadIdx.x;
        float acc = prm.s.p[0][e];
        for (int n = 1; n < prm.n_nodes; ++n) acc += prm.s.p[n][e];
        prm.out[e] = acc;
    }
}

// ---- quantizer ------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

// A group of KP = 2^m >= k adjacent lanes owns one compressed slice; lane j of the group owns
// coordinate j.  Every floating-point step is a single correctly rounded fp32 operation
// (explicit _rn intrinsics keep the compiler from fusing a multiply into an add), and the
// sum of squares runs as an xor-butterfly over the group, so the integer levels are a pure
// function of the input bits.
template <int KP>
__global__ void __launch_bounds__(256) quantize_kernel(int k, int64_t S, const float *__restrict__ s_node,
                                                       int levels, uint64_t seed, uint32_t node,
                                                       int8_t *__restrict__ q, float *__restrict__ norms)
{
    constexpr int GROUPS = 256 / KP;
    const int j = threadIdx.x % KP;
    const int grp = threadIdx.x / KP;
    const uint64_t hnode = mix64(seed + 0x9E3779B97F4A7C15ULL * ((uint64_t)node + 1ULL));
    const float fl = (float)levels;
    for (int64_t base = (int64_t)blockIdx.x * GROUPS; base < S; base += (int64_t)gridDim.x * GROUPS) {
        const int64_t i = base + grp;  // the whole warp stays in the loop: shuffles need every lane
        const bool live = i < S && j < k;
        const float v = live ? s_node[i * k + j] : 0.0f;
        float a = __fmul_rn(v, v);
#pragma unroll
        for (int stride = KP / 2; stride >= 1; stride /= 2)
            a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, stride));
        const float norm = __fsqrt_rn(a);
        int level = 0;
        if (norm > 0.0f) {
            const float r = __fmul_rn(fabsf(v), __fdiv_rn(fl, norm));
            const float lo = floorf(r);
            const float p = __fsub_rn(r, lo);
            const uint64_t h = mix64(hnode ^ (0xD1B54A32D192ED03ULL * ((uint64_t)i + 1ULL)));
            uint32_t x = (uint32_t)(h >> 32) ^ ((uint32_t)h + 0x9E3779B9u * ((uint32_t)j + 1u));
            x ^= x >> 16; x *= 0x7FEB352Du;
            x ^= x >> 15; x *= 0x846CA68Bu;
            x ^= x >> 16;
            const float u = __fmul_rn((float)(x >> 8), 1.0f / 16777216.0f);
            level = (int)lo + ((u < p) ? 1 : 0);
            level = min(level, levels);
        }
        if (live) {
            q[i * k + j] = (int8_t)((v < 0.0f) ? -level : level);
            if (j == 0) norms[i] = norm;
        }
    }
}

struct QaggParams {
    int n_nodes, k, levels;
    int64_t S;
    uint64_t seed;
    NodePtrs<const float> s;
    NodePtrs<int8_t> q;       // optional outputs (NULL entries when not wanted)
    NodePtrs<float> norms;
    float *out;
};

// Every node's compressed vectors quantized and the dequantised vectors summed, in one launch: the group of
// KP lanes that owns a slice walks the nodes in order, quantizes s_{n,i} exactly as quantize_kernel does and
// adds q * (norm / levels) to its running sum.
template <int KP>
__global__ void __launch_bounds__(256) quantize_aggregate_kernel(const __grid_constant__ QaggParams prm)
{
    constexpr int GROUPS = 256 / KP;
    __shared__ uint64_t node_hash[GVQ_MAX_NODES];   // the (seed, node) half of the hash, the same for every slice
    if (threadIdx.x < prm.n_nodes)
        node_hash[threadIdx.x] = mix64(prm.seed + 0x9E3779B97F4A7C15ULL * ((uint64_t)threadIdx.x + 1ULL));
    __syncthreads();
    const int j = threadIdx.x % KP;
    const int grp = threadIdx.x / KP;
    const int k = prm.k;
    const float fl = (float)prm.levels;
    const uint32_t jmix = 0x9E3779B9u * ((uint32_t)j + 1u);
    for (int64_t base = (int64_t)blockIdx.x * GROUPS; base < prm.S; base += (int64_t)gridDim.x * GROUPS) {
        const int64_t i = base + grp;
        const bool live = i < prm.S && j < k;
        const uint64_t slice_key = 0xD1B54A32D192ED03ULL * ((uint64_t)i + 1ULL);
        float acc = 0.0f;
#pragma unroll 4
        for (int n = 0; n < prm.n_nodes; ++n) {
            const float v = live ? __ldcs(prm.s.p[n] + i * k + j) : 0.0f;
            float a = __fmul_rn(v, v);
#pragma unroll
            for (int stride = KP / 2; stride >= 1; stride /= 2)
                a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, stride));
            const float norm = __fsqrt_rn(a);
            const float norm_div = norm > 0.0f ? norm : 1.0f;   // a zero vector quantizes to level 0 either way
            const float r = __fmul_rn(fabsf(v), __fdiv_rn(fl, norm_div));
            // floor, int <-> float conversions through the 2^23 trick (exact for these small magnitudes; they
            // keep the work on the FP32 / integer pipes instead of the conversion unit)
            float lo = __fsub_rn(__fadd_rn(r, 8388608.0f), 8388608.0f);   // r rounded to nearest, 0 <= r <= levels
            if (lo > r) lo = __fsub_rn(lo, 1.0f);
            const int ilo = __float_as_int(__fadd_rn(lo, 8388608.0f)) - 0x4B000000;
            const float p = __fsub_rn(r, lo);
            const uint64_t h = mix64(node_hash[n] ^ slice_key);
            uint32_t x = (uint32_t)(h >> 32) ^ ((uint32_t)h + jmix);
            x ^= x >> 16; x *= 0x7FEB352Du;
            x ^= x >> 15; x *= 0x846CA68Bu;
            x ^= x >> 16;
            // (float)(x >> 8): low 23 bits by the same trick, bit 23 added back (the sum is < 2^24, exact)
            float m = __fsub_rn(__int_as_float(0x4B000000 | ((x >> 8) & 0x7FFFFF)), 8388608.0f);
            if (x & 0x80000000u) m = __fadd_rn(m, 8388608.0f);
            const float u = __fmul_rn(m, 1.0f / 16777216.0f);
            const int level = norm > 0.0f ? min(ilo + ((u < p) ? 1 : 0), prm.levels) : 0;
            const int qv = (v < 0.0f) ? -level : level;
            const float qf = __fsub_rn(__int_as_float(0x4B400000 + qv), 12582912.0f);   // (float)qv, |qv| <= 127
            if (live) {
                if (prm.q.p[n]) prm.q.p[n][i * k + j] = (int8_t)qv;
                if (j == 0 && prm.norms.p[n]) prm.norms.p[n][i] = norm;
            }
            acc += __fmul_rn(qf, __fdiv_rn(norm, fl));
        }
        if (live) prm.out[i * k + j] = acc;
    }
}

struct DeqParams {
    int n_nodes, k, levels;
    int64_t S;
    NodePtrs<const int8_t> q;
    NodePtrs<const float> norms;
    float *out;
};

// out[i][j] = sum_n q_n[i][j] * (norm_n[i] / levels), node order.
__global__ void __launch_bounds__(256) dequantize_aggregate_kernel(const __grid_constant__ DeqParams prm)
{
    const int64_t total = prm.S * prm.k;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const float fl = (float)prm.levels;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        const int64_t i = e / prm.k;
        float acc = 0.0f;
        for (int n = 0; n < prm.n_nodes; ++n)
            acc += __fmul_rn((float)prm.q.p[n][e], __fdiv_rn(prm.norms.p[n][i], fl));
        prm.out[e] = acc;
    }
}

int grid_for(int64_t work_items, int per_block, int num_sms, int waves)
{
    int64_t blocks = (work_items + per_block - 1) / per_block;
    const int64_t cap = (int64_t)num_sms * waves;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace

cudaError_t launch_aggregate(cudaStream_t st, int num_sms, const NodePtrs<const float> &s, int n_nodes,
                             int64_t count, float *out)
{
    if (count == 0) return cudaSuccess;
    AggParams prm;
    prm.n_nodes = n_nodes; prm.count = count; prm.s = s; prm.out = out;
    aggregate_kernel<<<grid_for(count / 4 + 1, 256, num_sms, 8), 256, 0, st>>>(prm);
    return cudaGetLastError();
}

cudaError_t launch_quantize(cudaStream_t st, int k, int64_t S, const float *s_node, int levels,
                            uint64_t seed, uint32_t node, int8_t *q, float *norms)
{
    if (S == 0) return cudaSuccess;
    int kp = 1;
    while (kp < k) kp <<= 1;
    const int groups = 256 / kp;
    int64_t blocks = (S + groups - 1) / groups;
    if (blocks > 148 * 16) blocks = 148 * 16;
    const int grid = (int)blocks;
    switch (kp) {
    case 1: quantize_kernel<1><<<grid, 256, 0, st>>>(k, S, s_node, levels, seed, node, q, norms); break;
    case 2: quantize_kernel<2><<<grid, 256, 0, st>>>(k, S, s_node, levels, seed, node, q, norms); break;
    case 4: quantize_kernel<4><<<grid, 256, 0, st>>>(k, S, s_node, levels, seed, node, q, norms); break;
    case 8: quantize_kernel<8><<<grid, 256, 0, st>>>(k, S, s_node, levels, seed, node, q, norms); break;
    case 16: quantize_kernel<16><<<grid, 256, 0, st>>>(k, S, s_node, levels, seed, node, q, norms); break;
    case 32: quantize_kernel<32><<<grid, 256, 0, st>>>(k, S, s_node, levels, seed, node, q, norms); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_aggregate(cudaStream_t st, int num_sms, int k, int64_t S, const NodePtrs<const float> &s,
                                      int n_nodes, int levels, uint64_t seed, const NodePtrs<int8_t> &q,
                                      const NodePtrs<float> &norms, float *s_sum)
{
    if (S == 0) return cudaSuccess;
    QaggParams prm;
    prm.n_nodes = n_nodes; prm.k = k; prm.levels = levels; prm.S = S; prm.seed = seed;
    prm.s = s; prm.q = q; prm.norms = norms; prm.out = s_sum;
    int kp = 1;
    while (kp < k) kp <<= 1;
    const int groups = 256 / kp;
    int64_t blocks = (S + groups - 1) / groups;
    if (blocks > (int64_t)num_sms * 16) blocks = (int64_t)num_sms * 16;
    const int grid = (int)blocks;
    switch (kp) {
    case 1: quantize_aggregate_kernel<1><<<grid, 256, 0, st>>>(prm); break;
    case 2: quantize_aggregate_kernel<2><<<grid, 256, 0, st>>>(prm); break;
    case 4: quantize_aggregate_kernel<4><<<grid, 256, 0, st>>>(prm); break;
    case 8: quantize_aggregate_kernel<8><<<grid, 256, 0, st>>>(prm); break;
    case 16: quantize_aggregate_kernel<16><<<grid, 256, 0, st>>>(prm); break;
    case 32: quantize_aggregate_kernel<32><<<grid, 256, 0, st>>>(prm); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_dequantize_aggregate(cudaStream_t st, int num_sms, int k, int64_t S,
                                        const NodePtrs<const int8_t> &q, const NodePtrs<const float> &norms,
                                        int n_nodes, int levels, float *s_sum)
{
    if (S == 0) return cudaSuccess;
    DeqParams prm;
    prm.n_nodes = n_nodes; prm.k = k; prm.levels = levels; prm.S = S; prm.q = q; prm.norms = norms;
    prm.out = s_sum;
    dequantize_aggregate_kernel<<<grid_for(S * k, 256, num_sms, 8), 256, 0, st>>>(prm);
    return cudaGetLastError();
}

}  // namespace gvq
