// Compressed-domain aggregation on materialised buffers (Eq. 4) and the stochastic scalar
// quantizer of compressed vectors with its dequantise-and-sum counterpart.
#include "gvq_internal.h"
#include "quantizer.cuh"

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
using quant::mix64;

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

// ---- the same with one thread per bucket (k = 4, 8, 16 or 32 exactly) --------------------------
// A warp takes 32 consecutive slices: their 32 k floats are read coalesced, passed through a padded
// shared-memory tile so that every thread ends up with its own slice in registers, and quantized by
// quantize_bucket -- the per-bucket work once per slice instead of once per lane.
constexpr int ROW_WARPS = 8;

template <int KP>
__device__ __forceinline__ void load_rows(float *tile, const float *__restrict__ src, int64_t slice0, int64_t S, int lane,
                                          float (&v)[KP])
{
    constexpr int LD = KP + 4;       // row pitch in floats: a quarter-warp's 128-bit reads cover all 32 banks
    constexpr int F4 = KP / 4;       // 128-bit words per row
#pragma unroll
    for (int it = 0; it < F4; ++it) {
        const int f = it * 32 + lane, row = f / F4, c4 = f - row * F4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (slice0 + row < S) x = __ldcs(reinterpret_cast<const float4 *>(src + (slice0 + row) * KP) + c4);
        *reinterpret_cast<float4 *>(tile + row * LD + c4 * 4) = x;
    }
    __syncwarp();
#pragma unroll
    for (int c4 = 0; c4 < F4; ++c4) {
        const float4 x = *reinterpret_cast<const float4 *>(tile + lane * LD + c4 * 4);
        v[4 * c4] = x.x; v[4 * c4 + 1] = x.y; v[4 * c4 + 2] = x.z; v[4 * c4 + 3] = x.w;
    }
    __syncwarp();
}

template <int KP>
__device__ __forceinline__ void store_levels(int8_t *q, int64_t slice, const uint32_t (&packed)[KP / 4])
{
    uint32_t *dst = reinterpret_cast<uint32_t *>(q + slice * KP);
    if constexpr (KP >= 16) {
#pragma unroll
        for (int w = 0; w < KP / 16; ++w)
            reinterpret_cast<uint4 *>(dst)[w] = make_uint4(packed[4 * w], packed[4 * w + 1], packed[4 * w + 2], packed[4 * w + 3]);
    } else if constexpr (KP == 8) {
        *reinterpret_cast<uint2 *>(dst) = make_uint2(packed[0], packed[1]);
    } else {
        dst[0] = packed[0];
    }
}

template <int KP>
__global__ void __launch_bounds__(ROW_WARPS * 32) quantize_rows_kernel(int64_t S, const float *__restrict__ s_node,
                                                                        int levels, uint64_t seed, uint32_t node,
                                                                        int8_t *__restrict__ q, float *__restrict__ norms)
{
    __shared__ __align__(16) float tiles[ROW_WARPS][32 * (KP + 4)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t hnode = quant::node_key(seed, node);
    const int64_t step = (int64_t)gridDim.x * ROW_WARPS * 32;
    for (int64_t slice0 = ((int64_t)blockIdx.x * ROW_WARPS + warp) * 32; slice0 < S; slice0 += step) {
        float v[KP], unused[KP];
        uint32_t packed[KP / 4];
#pragma unroll
        for (int j = 0; j < KP; ++j) unused[j] = 0.0f;
        load_rows<KP>(tiles[warp], s_node, slice0, S, lane, v);
        const int64_t i = slice0 + lane;
        const float norm = quant::quantize_bucket<KP>(v, levels, hnode, i, packed, unused);
        if (i < S) {
            store_levels<KP>(q, i, packed);
            norms[i] = norm;
        }
    }
}

template <int KP>
__global__ void __launch_bounds__(ROW_WARPS * 32) quantize_aggregate_rows_kernel(const __grid_constant__ QaggParams prm)
{
    __shared__ __align__(16) float tiles[ROW_WARPS][32 * (KP + 4)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t step = (int64_t)gridDim.x * ROW_WARPS * 32;
    for (int64_t slice0 = ((int64_t)blockIdx.x * ROW_WARPS + warp) * 32; slice0 < prm.S; slice0 += step) {
        const int64_t i = slice0 + lane;
        float acc[KP];
#pragma unroll
        for (int j = 0; j < KP; ++j) acc[j] = 0.0f;
        for (int n = 0; n < prm.n_nodes; ++n) {
            float v[KP];
            uint32_t packed[KP / 4];
            load_rows<KP>(tiles[warp], prm.s.p[n], slice0, prm.S, lane, v);
            const float norm = quant::quantize_bucket<KP>(v, prm.levels, quant::node_key(prm.seed, (uint32_t)n), i, packed, acc);
            if (i < prm.S) {
                if (prm.q.p[n]) store_levels<KP>(prm.q.p[n], i, packed);
                if (prm.norms.p[n]) prm.norms.p[n][i] = norm;
            }
        }
        if (i < prm.S) {
#pragma unroll
            for (int c4 = 0; c4 < KP / 4; ++c4)
                reinterpret_cast<float4 *>(prm.out + i * KP)[c4] =
                    make_float4(acc[4 * c4], acc[4 * c4 + 1], acc[4 * c4 + 2], acc[4 * c4 + 3]);
        }
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

// The same for k a multiple of 4: a thread owns four adjacent coordinates of one slice (one 32-bit load of
// levels, one division per node, one 128-bit store).
__global__ void __launch_bounds__(256) dequantize_aggregate4_kernel(const __grid_constant__ DeqParams prm)
{
    const int k4 = prm.k / 4;
    const int64_t total = prm.S * k4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const float fl = (float)prm.levels;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        const int64_t i = e / k4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int n = 0; n < prm.n_nodes; ++n) {
            const uint32_t w = __ldcs(reinterpret_cast<const uint32_t *>(prm.q.p[n]) + e);
            const float step = __fdiv_rn(__ldg(prm.norms.p[n] + i), fl);
            acc.x += __fmul_rn((float)(int8_t)(w & 0xff), step);
            acc.y += __fmul_rn((float)(int8_t)((w >> 8) & 0xff), step);
            acc.z += __fmul_rn((float)(int8_t)((w >> 16) & 0xff), step);
            acc.w += __fmul_rn((float)(int8_t)(w >> 24), step);
        }
        reinterpret_cast<float4 *>(prm.out)[e] = acc;
    }
}

// ---- Eq. 7's two sums from materialised buffers (shapes without a tensor-core projection) -----------------
// grid (tiles of 256 slices, nodes); a warp takes a slice at a time: sum (x - mu / N)^2 over its d entries and
// sum s^2 over its k compressed values; one double atomic per CTA and sum.
struct MonParams {
    int d, k, n_nodes, mean_div;
    const int32_t *tile_layer, *tile_row0;
    const int64_t *layer_off, *layer_soff;
    const int32_t *layer_S;
    const float *mu;
    NodePtrs<const float> g;
    NodePtrs<const float> s;
    double *monitor;
};

__global__ void __launch_bounds__(256) monitor_kernel(const __grid_constant__ MonParams prm)
{
    __shared__ float red[2][8];
    const int tile = blockIdx.x, node = blockIdx.y;
    const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile];
    const int count = min(kProjectRows, prm.layer_S[layer] - row0);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float *x = prm.g.p[node] + prm.layer_off[layer] + (int64_t)row0 * prm.d;
    const float *sv = prm.s.p[node] + (prm.layer_soff[layer] + row0) * (int64_t)prm.k;
    const float *m = prm.mu + (size_t)layer * prm.d;
    const float div = (float)prm.mean_div;
    float e = 0.0f, c = 0.0f;
    for (int r = warp; r < count; r += 8) {
        for (int t = lane; t < prm.d; t += 32) {
            const float v = x[(size_t)r * prm.d + t] - m[t] / div;
            e = fmaf(v, v, e);
        }
        for (int j = lane; j < prm.k; j += 32) {
            const float v = sv[(size_t)r * prm.k + j];
            c = fmaf(v, v, c);
        }
    }
    for (int o = 16; o >= 1; o >>= 1) {
        e += __shfl_xor_sync(0xffffffffu, e, o);
        c += __shfl_xor_sync(0xffffffffu, c, o);
    }
    if (lane == 0) { red[0][warp] = e; red[1][warp] = c; }
    __syncthreads();
    if (threadIdx.x < 2) {
        double tot = 0.0;
        for (int w = 0; w < 8; ++w) tot += (double)red[threadIdx.x][w];
        atomicAdd(prm.monitor + ((size_t)layer * 2 + threadIdx.x) * prm.n_nodes + node, tot);
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

cudaError_t launch_monitor(cudaStream_t st, int d, int k, const TileTable &tiles, const LayerTables &lt,
                           const NodePtrs<const float> &g, const NodePtrs<const float> &s, int n_nodes, int mean_div,
                           const float *mu, double *monitor)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    MonParams prm;
    prm.d = d; prm.k = k; prm.n_nodes = n_nodes; prm.mean_div = mean_div;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.layer_S = lt.S;
    prm.mu = mu; prm.g = g; prm.s = s; prm.monitor = monitor;
    monitor_kernel<<<dim3(tiles.n_tiles, n_nodes), 256, 0, st>>>(prm);
    return cudaGetLastError();
}

cudaError_t launch_quantize(cudaStream_t st, int num_sms, int k, int64_t S, const float *s_node, int levels,
                            uint64_t seed, uint32_t node, int8_t *q, float *norms)
{
    if (S == 0) return cudaSuccess;
    if (k == 4 || k == 8 || k == 16 || k == 32) {   // one thread per bucket
        const int grid = grid_for(S, ROW_WARPS * 32, num_sms, 8);
        switch (k) {
        case 4: quantize_rows_kernel<4><<<grid, ROW_WARPS * 32, 0, st>>>(S, s_node, levels, seed, node, q, norms); break;
        case 8: quantize_rows_kernel<8><<<grid, ROW_WARPS * 32, 0, st>>>(S, s_node, levels, seed, node, q, norms); break;
        case 16: quantize_rows_kernel<16><<<grid, ROW_WARPS * 32, 0, st>>>(S, s_node, levels, seed, node, q, norms); break;
        default: quantize_rows_kernel<32><<<grid, ROW_WARPS * 32, 0, st>>>(S, s_node, levels, seed, node, q, norms); break;
        }
        return cudaGetLastError();
    }
    int kp = 1;
    while (kp < k) kp <<= 1;
    const int groups = 256 / kp;
    int64_t blocks = (S + groups - 1) / groups;
    if (blocks > (int64_t)num_sms * 16) blocks = (int64_t)num_sms * 16;
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
    if (k == 4 || k == 8 || k == 16 || k == 32) {   // one thread per bucket
        const int grid = grid_for(S, ROW_WARPS * 32, num_sms, 8);
        switch (k) {
        case 4: quantize_aggregate_rows_kernel<4><<<grid, ROW_WARPS * 32, 0, st>>>(prm); break;
        case 8: quantize_aggregate_rows_kernel<8><<<grid, ROW_WARPS * 32, 0, st>>>(prm); break;
        case 16: quantize_aggregate_rows_kernel<16><<<grid, ROW_WARPS * 32, 0, st>>>(prm); break;
        default: quantize_aggregate_rows_kernel<32><<<grid, ROW_WARPS * 32, 0, st>>>(prm); break;
        }
        return cudaGetLastError();
    }
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
    if (k % 4 == 0)
        dequantize_aggregate4_kernel<<<grid_for(S * (k / 4), 256, num_sms, 8), 256, 0, st>>>(prm);
    else
        dequantize_aggregate_kernel<<<grid_for(S * k, 256, num_sms, 8), 256, 0, st>>>(prm);
    return cudaGetLastError();
}

}  // namespace gvq
