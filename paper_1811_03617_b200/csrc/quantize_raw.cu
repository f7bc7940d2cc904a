// The stochastic quantizer applied to RAW gradient slices, 4 bits per entry (Section 3: the iterations that
// aggregate without the PCA compressor send quantized gradients; the experiments use 4-bit QSGD).  Bucket = one
// slice of d entries, arithmetic exactly as gvq_quantize defines it with k := d and the global slice index as
// counter; levels <= 7 are packed two per byte (two's-complement nibbles, even entry low).
//
// A warp owns a slice: entry j sits in register j / 32 of lane j % 32, so the strides >= 32 of the butterfly sum
// pair registers of one lane and the strides < 32 are shuffles -- the same additions, in the same order, as the
// definition's full-width butterfly.
#include "gvq_internal.h"
#include "quantizer.cuh"

namespace gvq {
namespace {

struct RawParams {
    int d, levels, n_nodes;
    uint64_t seed;
    uint32_t node;
    const int32_t *tile_layer, *tile_row0, *layer_S;
    const int64_t *layer_off, *layer_soff;
    const float *g;
    uint8_t *q4;
    float *norms;
};

// R = registers per lane = max(1, kp / 32), kp = next power of two >= d.  grid = tiles of 256 slices, 8 warps.
template <int R>
__global__ void __launch_bounds__(256) quantize_raw4_kernel(const __grid_constant__ RawParams prm)
{
    __shared__ int8_t lv[8][32 * R];
    const int tile = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile], d = prm.d;
    const int count = min(kProjectRows, prm.layer_S[layer] - row0);
    const float fl = (float)prm.levels;
    const uint64_t hnode = quant::node_key(prm.seed, prm.node);
    int kp = 1;
    while (kp < d) kp <<= 1;
    for (int r = warp; r < count; r += 8) {
        const int64_t gslice = prm.layer_soff[layer] + row0 + r;
        const float *x = prm.g + prm.layer_off[layer] + (int64_t)(row0 + r) * d;
        float v[R], a[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int j = 32 * i + lane;
            v[i] = j < d ? __ldcs(x + j) : 0.0f;
            a[i] = __fmul_rn(v[i], v[i]);
        }
        // strides kp / 2 ... 32: registers of one lane;  a[i] <- a[i] + a[i ^ s] for all i at once
#pragma unroll
        for (int s = R / 2; s >= 1; s >>= 1) {
            float b[R];
#pragma unroll
            for (int i = 0; i < R; ++i) b[i] = __fadd_rn(a[i], a[i ^ s]);
#pragma unroll
            for (int i = 0; i < R; ++i) a[i] = b[i];
        }
        float tot = a[0];
        for (int s = min(16, kp / 2); s >= 1; s >>= 1) tot = __fadd_rn(tot, __shfl_xor_sync(0xffffffffu, tot, s));
        const float norm = __fsqrt_rn(__shfl_sync(0xffffffffu, tot, 0));
        const float scale = norm > 0.0f ? __fdiv_rn(fl, norm) : 0.0f;
        const uint64_t hs = quant::mix64(hnode ^ (0xD1B54A32D192ED03ULL * ((uint64_t)gslice + 1ULL)));
        const uint32_t h_hi = (uint32_t)(hs >> 32), h_lo = (uint32_t)hs;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int j = 32 * i + lane;
            const float rr = __fmul_rn(fabsf(v[i]), scale);
            const float lo = floorf(rr);
            const float pr = __fsub_rn(rr, lo);
            const float u = __fmul_rn((float)quant::coord_hash24(h_hi, h_lo, (uint32_t)j), 1.0f / 16777216.0f);
            int level = min((int)lo + ((u < pr) ? 1 : 0), prm.levels);
            level = v[i] < 0.0f ? -level : level;
            lv[warp][j] = (int8_t)level;
        }
        __syncwarp();
        // pack: four bytes (eight entries) per store where a slice's bytes stay 4-byte aligned (d % 8 == 0)
        uint8_t *dst = prm.q4 + gslice * (d / 2);
        auto byte_of = [&](int b) {
            return (uint32_t)lv[warp][2 * b] & 0xFu | (((uint32_t)lv[warp][2 * b + 1] & 0xFu) << 4);
        };
        if (d % 8 == 0) {
            for (int w4 = lane; w4 < d / 8; w4 += 32)
                reinterpret_cast<uint32_t *>(dst)[w4] = byte_of(4 * w4) | (byte_of(4 * w4 + 1) << 8) |
                                                        (byte_of(4 * w4 + 2) << 16) | (byte_of(4 * w4 + 3) << 24);
        } else {
            for (int b = lane; b < d / 2; b += 32) dst[b] = (uint8_t)byte_of(b);
        }
        if (lane == 0) prm.norms[gslice] = norm;
        __syncwarp();
    }
}

// All N nodes in one launch: a warp takes a slice through the nodes in order, quantizes each node's copy as above
// and keeps the sum of the dequantised values in registers; q4 / norms of the nodes are optional outputs.
struct RawAggParams {
    int d, levels, n_nodes;
    uint64_t seed;
    const int32_t *tile_layer, *tile_row0, *layer_S;
    const int64_t *layer_off, *layer_soff;
    NodePtrs<const float> g;
    NodePtrs<uint8_t> q4;
    NodePtrs<float> norms;
    float *out;
};

template <int R>
__global__ void __launch_bounds__(256) quantize_raw4_aggregate_kernel(const __grid_constant__ RawAggParams prm)
{
    __shared__ int8_t lv[8][32 * R];
    __shared__ uint64_t node_hash[GVQ_MAX_NODES];
    const int tile = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile], d = prm.d;
    const int count = min(kProjectRows, prm.layer_S[layer] - row0);
    const float fl = (float)prm.levels;
    if (threadIdx.x < prm.n_nodes) node_hash[threadIdx.x] = quant::node_key(prm.seed, (uint32_t)threadIdx.x);
    __syncthreads();
    int kp = 1;
    while (kp < d) kp <<= 1;
    const int s0 = min(16, kp / 2);
    for (int r = warp; r < count; r += 8) {
        const int64_t gslice = prm.layer_soff[layer] + row0 + r;
        const int64_t goff = prm.layer_off[layer] + (int64_t)(row0 + r) * d;
        const uint64_t slice_key = 0xD1B54A32D192ED03ULL * ((uint64_t)gslice + 1ULL);
        float acc[R];
        uint32_t jc[R];
#pragma unroll
        for (int i = 0; i < R; ++i) { acc[i] = 0.0f; jc[i] = 0x9E3779B9u * ((uint32_t)(32 * i + lane) + 1u); }
        float vn[R];   // the next node's entries, loaded one node ahead
#pragma unroll
        for (int i = 0; i < R; ++i) vn[i] = (32 * i + lane) < d ? __ldcs(prm.g.p[0] + goff + 32 * i + lane) : 0.0f;
        for (int n = 0; n < prm.n_nodes; ++n) {
            float v[R], a[R];
#pragma unroll
            for (int i = 0; i < R; ++i) { v[i] = vn[i]; a[i] = __fmul_rn(v[i], v[i]); }
            if (n + 1 < prm.n_nodes) {
#pragma unroll
                for (int i = 0; i < R; ++i) vn[i] = (32 * i + lane) < d ? __ldcs(prm.g.p[n + 1] + goff + 32 * i + lane) : 0.0f;
            }
#pragma unroll
            for (int s = R / 2; s >= 1; s >>= 1) {
                float b[R];
#pragma unroll
                for (int i = 0; i < R; ++i) b[i] = __fadd_rn(a[i], a[i ^ s]);
#pragma unroll
                for (int i = 0; i < R; ++i) a[i] = b[i];
            }
            float tot = a[0];
            for (int s = s0; s >= 1; s >>= 1) tot = __fadd_rn(tot, __shfl_xor_sync(0xffffffffu, tot, s));
            const float norm = __fsqrt_rn(__shfl_sync(0xffffffffu, tot, 0));
            const float scale = norm > 0.0f ? __fdiv_rn(fl, norm) : 0.0f;
            const float step = __fdiv_rn(norm, fl);
            const uint64_t hs = quant::mix64(node_hash[n] ^ slice_key);
            const uint32_t h_hi = (uint32_t)(hs >> 32), h_lo = (uint32_t)hs;
            const bool emit = prm.q4.p[n] != nullptr;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                const float rr = __fmul_rn(fabsf(v[i]), scale);
                const float lo = floorf(rr);
                const float pr = __fsub_rn(rr, lo);
                uint32_t x = h_hi ^ (h_lo + jc[i]);   // coord_hash24 with the coordinate's multiple precomputed
                x ^= x >> 16; x *= 0x7FEB352Du;
                x ^= x >> 15; x *= 0x846CA68Bu;
                x ^= x >> 16;
                const float u = __fmul_rn((float)(x >> 8), 1.0f / 16777216.0f);
                // the level as a float (small integers are exact): no integer round trip unless it is written out
                const float lf = copysignf(fminf(lo + ((u < pr) ? 1.0f : 0.0f), fl), v[i]);
                acc[i] += __fmul_rn(lf, step);
                if (emit) lv[warp][32 * i + lane] = (int8_t)(int)lf;
            }
            if (emit) {
                __syncwarp();
                uint8_t *dst = prm.q4.p[n] + gslice * (d / 2);
                auto byte_of = [&](int b) {
                    return (uint32_t)lv[warp][2 * b] & 0xFu | (((uint32_t)lv[warp][2 * b + 1] & 0xFu) << 4);
                };
                if (d % 8 == 0) {
                    for (int w4 = lane; w4 < d / 8; w4 += 32)
                        reinterpret_cast<uint32_t *>(dst)[w4] = byte_of(4 * w4) | (byte_of(4 * w4 + 1) << 8) |
                                                                (byte_of(4 * w4 + 2) << 16) | (byte_of(4 * w4 + 3) << 24);
                } else {
                    for (int b = lane; b < d / 2; b += 32) dst[b] = (uint8_t)byte_of(b);
                }
                __syncwarp();
            }
            if (lane == 0 && prm.norms.p[n]) prm.norms.p[n][gslice] = norm;
        }
#pragma unroll
        for (int i = 0; i < R; ++i)
            if (32 * i + lane < d) prm.out[goff + 32 * i + lane] = acc[i];
    }
}

struct RawDeqParams {
    int d, levels, n_nodes;
    const int32_t *tile_layer, *tile_row0, *layer_S;
    const int64_t *layer_off, *layer_soff;
    NodePtrs<const uint8_t> q4;
    NodePtrs<const float> norms;
    float *out;
};

// out[slice entries] = sum_n q * (norm_n / levels), node order; a thread owns 4 adjacent entries (2 bytes) of a slice
__global__ void __launch_bounds__(256) dequantize_raw4_kernel(const __grid_constant__ RawDeqParams prm)
{
    const int tile = blockIdx.x;
    const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile], d = prm.d;
    const int count = min(kProjectRows, prm.layer_S[layer] - row0);
    const float fl = (float)prm.levels;
    const int d4 = d / 4;
    for (int e = threadIdx.x; e < count * d4; e += 256) {
        const int r = e / d4, c4 = e - r * d4;
        const int64_t gslice = prm.layer_soff[layer] + row0 + r;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int n = 0; n < prm.n_nodes; ++n) {
            const uint32_t w = *reinterpret_cast<const uint16_t *>(prm.q4.p[n] + gslice * (d / 2) + 2 * c4);
            const float step = __fdiv_rn(__ldg(prm.norms.p[n] + gslice), fl);
            auto nib = [](uint32_t x) { return (float)((int)(x ^ 8u) - 8); };   // two's-complement nibble
            acc.x += __fmul_rn(nib(w & 0xFu), step);
            acc.y += __fmul_rn(nib((w >> 4) & 0xFu), step);
            acc.z += __fmul_rn(nib((w >> 8) & 0xFu), step);
            acc.w += __fmul_rn(nib((w >> 12) & 0xFu), step);
        }
        *reinterpret_cast<float4 *>(prm.out + prm.layer_off[layer] + (int64_t)(row0 + r) * d + 4 * c4) = acc;
    }
}

// The same with 16 adjacent entries (8 bytes of levels) per thread, for d a multiple of 16: wider loads, and the
// loads of four nodes in flight together.
__global__ void __launch_bounds__(256) dequantize_raw4_wide_kernel(const __grid_constant__ RawDeqParams prm)
{
    const int tile = blockIdx.x;
    const int layer = prm.tile_layer[tile], row0 = prm.tile_row0[tile], d = prm.d;
    const int count = min(kProjectRows, prm.layer_S[layer] - row0);
    const float fl = (float)prm.levels;
    const int d16 = d / 16;
    for (int e = threadIdx.x; e < count * d16; e += 256) {
        const int r = e / d16, c16 = e - r * d16;
        const int64_t gslice = prm.layer_soff[layer] + row0 + r;
        float acc[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] = 0.0f;
        for (int n0 = 0; n0 < prm.n_nodes; n0 += 4) {
            uint2 w[4];
            float nrm[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (n0 + u < prm.n_nodes) {
                    w[u] = __ldcs(reinterpret_cast<const uint2 *>(prm.q4.p[n0 + u] + gslice * (d / 2)) + c16);
                    nrm[u] = __ldg(prm.norms.p[n0 + u] + gslice);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (n0 + u < prm.n_nodes) {   // nodes in ascending order, as defined
                    const float step = __fdiv_rn(nrm[u], fl);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint32_t word = i < 8 ? w[u].x : w[u].y;
                        const uint32_t nib = (word >> (4 * (i & 7))) & 0xFu;
                        // the signed level as a float without the conversion unit: 1.5 * 2^23 + level, minus 1.5 * 2^23
                        const float q = __int_as_float(0x4B400000 + (int)(nib ^ 8u) - 8) - 12582912.0f;
                        acc[i] += __fmul_rn(q, step);
                    }
                }
            }
        }
        float4 *dst = reinterpret_cast<float4 *>(prm.out + prm.layer_off[layer] + (int64_t)(row0 + r) * d + 16 * c16);
#pragma unroll
        for (int v = 0; v < 4; ++v) dst[v] = make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
    }
}

}  // namespace

cudaError_t launch_quantize_raw4(cudaStream_t st, int d, const TileTable &tiles, const LayerTables &lt, const float *g,
                                 int levels, uint64_t seed, uint32_t node, uint8_t *q4, float *norms)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    RawParams prm;
    prm.d = d; prm.levels = levels; prm.n_nodes = 1; prm.seed = seed; prm.node = node;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0; prm.layer_S = lt.S;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.g = g; prm.q4 = q4; prm.norms = norms;
    int kp = 1;
    while (kp < d) kp <<= 1;
    switch (kp <= 32 ? 1 : kp / 32) {
    case 1: quantize_raw4_kernel<1><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 2: quantize_raw4_kernel<2><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 4: quantize_raw4_kernel<4><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 8: quantize_raw4_kernel<8><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 16: quantize_raw4_kernel<16><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 32: quantize_raw4_kernel<32><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_raw4_aggregate(cudaStream_t st, int d, const TileTable &tiles, const LayerTables &lt,
                                           const NodePtrs<const float> &g, int n_nodes, int levels, uint64_t seed,
                                           const NodePtrs<uint8_t> &q4, const NodePtrs<float> &norms, float *out)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    RawAggParams prm;
    prm.d = d; prm.levels = levels; prm.n_nodes = n_nodes; prm.seed = seed;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0; prm.layer_S = lt.S;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.g = g; prm.q4 = q4; prm.norms = norms; prm.out = out;
    int kp = 1;
    while (kp < d) kp <<= 1;
    switch (kp <= 32 ? 1 : kp / 32) {
    case 1: quantize_raw4_aggregate_kernel<1><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 2: quantize_raw4_aggregate_kernel<2><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 4: quantize_raw4_aggregate_kernel<4><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 8: quantize_raw4_aggregate_kernel<8><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 16: quantize_raw4_aggregate_kernel<16><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    case 32: quantize_raw4_aggregate_kernel<32><<<tiles.n_tiles, 256, 0, st>>>(prm); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_dequantize_raw4(cudaStream_t st, int d, const TileTable &tiles, const LayerTables &lt,
                                   const NodePtrs<const uint8_t> &q4, const NodePtrs<const float> &norms, int n_nodes,
                                   int levels, float *out)
{
    if (tiles.n_tiles == 0) return cudaSuccess;
    RawDeqParams prm;
    prm.d = d; prm.levels = levels; prm.n_nodes = n_nodes;
    prm.tile_layer = tiles.layer; prm.tile_row0 = tiles.row0; prm.layer_S = lt.S;
    prm.layer_off = lt.off; prm.layer_soff = lt.soff; prm.q4 = q4; prm.norms = norms; prm.out = out;
    if (d % 16 == 0) dequantize_raw4_wide_kernel<<<tiles.n_tiles, 256, 0, st>>>(prm);
    else dequantize_raw4_kernel<<<tiles.n_tiles, 256, 0, st>>>(prm);
    return cudaGetLastError();
}

}  // namespace gvq
