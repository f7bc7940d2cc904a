// The stochastic quantizer of one bucket (one compressed slice of one node) held in the registers of
// one thread, as gvq_quantize defines it: every floating-point step is one correctly rounded fp32
// operation (the _rn intrinsics keep the compiler from contracting a multiply into an add), the sum of
// squares is the xor-butterfly written out as its tree, the uniform comes from the stateless hash.
// With a whole bucket in one thread the per-bucket work (norm, square root, the two divisions, the
// 64-bit half of the hash) is done once, and a coordinate costs about 25 instructions.
#pragma once
#include <stdint.h>

namespace gvq {
namespace quant {

__device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

// the (seed, node) half of the hash: the same for every slice of a node
__device__ __forceinline__ uint64_t node_key(uint64_t seed, uint32_t node)
{
    return mix64(seed + 0x9E3779B97F4A7C15ULL * ((uint64_t)node + 1ULL));
}

// hash24(seed, node, slice, j) given h = mix64(node_key ^ slice term)
__device__ __forceinline__ uint32_t coord_hash24(uint32_t h_hi, uint32_t h_lo, uint32_t j)
{
    uint32_t x = h_hi ^ (h_lo + 0x9E3779B9u * (j + 1u));
    x ^= x >> 16; x *= 0x7FEB352Du;
    x ^= x >> 15; x *= 0x846CA68Bu;
    x ^= x >> 16;
    return x >> 8;
}

// The norm of a bucket from the first level of its butterfly: t[j] = v_j^2 + v_{j + KP/2}^2 (each square and each
// sum one rounded operation), j < KP / 2.  The remaining levels (strides KP / 4 .. 1) are taken here.
template <int HALF>
__device__ __forceinline__ float norm_from_first_level(float (&t)[HALF])
{
#pragma unroll
    for (int stride = HALF / 2; stride >= 1; stride >>= 1)
#pragma unroll
        for (int j = 0; j < stride; ++j) t[j] = __fadd_rn(t[j], t[j + stride]);
    return __fsqrt_rn(t[0]);
}

// What the coordinates of one bucket share: the slice's half of the hash and the two quotients of the norm.
struct BucketKeys {
    uint32_t h_hi, h_lo;
    float scale, step;   // levels / norm (0 when the norm is 0), norm / levels
    int levels;
};
__device__ __forceinline__ BucketKeys bucket_keys(float norm, int levels, uint64_t hnode, int64_t slice)
{
    BucketKeys k;
    const float fl = (float)levels;
    const uint64_t hs = mix64(hnode ^ (0xD1B54A32D192ED03ULL * ((uint64_t)slice + 1ULL)));
    k.h_hi = (uint32_t)(hs >> 32);
    k.h_lo = (uint32_t)hs;
    // norm == 0 (all v_j zero, or their squares underflowed): scale 0 gives r = 0, p = 0 and level 0, as defined
    k.scale = norm > 0.0f ? __fdiv_rn(fl, norm) : 0.0f;
    k.step = __fdiv_rn(norm, fl);
    k.levels = levels;
    return k;
}

// Quantizes the coordinates j0 .. j0 + C - 1 of a bucket (C a multiple of 4; the hash takes the coordinate's index
// in the whole bucket).  acc[i] += q * (norm / levels), the dequantised value; with PACK, packed[i / 4] receives the
// signed int8 levels, little end first.  Eight coordinates are taken through each step together so that their
// dependent chains overlap.
// The arithmetic is the definition's, value for value, written with operations that cost one issue slot of the
// FP32 pipe each wherever the definition allows it (the integer / conversion pipe has half the rate and the hash
// already fills it):
//   floor(r): r < 2^22, so t = r + 2^23 rounded DOWN is 2^23 + floor(r) exactly and floor(r) = t - 2^23 (exact);
//   u < p  with u = hash * 2^-24  <=>  float(hash) < p * 2^24 (both scalings by a power of two are exact);
//   the level stays a float: lo + (0 or 1), min with levels, the sign copied from v -- each of these values is an
//   integer of at most 7 bits, so the float holds exactly what the int8 code holds, and q * step is the same product.
template <int C, bool PACK = true>
__device__ __forceinline__ void quantize_columns(const float (&v)[C], int j0, const BucketKeys &k, uint32_t (&packed)[C / 4],
                                                 float (&acc)[C])
{
    constexpr int G = C < 8 ? C : 8;
    const float fl = (float)k.levels;
#pragma unroll
    for (int jb = 0; jb < C; jb += G) {
        float rr[G], hf[G], lv[G];
#pragma unroll
        for (int i = 0; i < G; ++i) rr[i] = __fmul_rn(fabsf(v[jb + i]), k.scale);
#pragma unroll
        for (int i = 0; i < G; ++i) hf[i] = __uint2float_rn(coord_hash24(k.h_hi, k.h_lo, (uint32_t)(j0 + jb + i)));
#pragma unroll
        for (int i = 0; i < G; ++i) {
            const float lo = __fsub_rn(__fadd_rd(rr[i], 8388608.0f), 8388608.0f);
            const float pr = __fsub_rn(rr[i], lo);
            const float up = hf[i] < __fmul_rn(pr, 16777216.0f) ? 1.0f : 0.0f;
            lv[i] = copysignf(fminf(__fadd_rn(lo, up), fl), v[jb + i]);
        }
#pragma unroll
        for (int i = 0; i < G; ++i) acc[jb + i] += __fmul_rn(lv[i], k.step);
        if constexpr (PACK) {
#pragma unroll
            for (int i = 0; i < G; i += 4) {
                const int q0 = __float2int_rn(lv[i]), q1 = __float2int_rn(lv[i + 1]);
                const int q2 = __float2int_rn(lv[i + 2]), q3 = __float2int_rn(lv[i + 3]);
                packed[(jb + i) / 4] = (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) |
                                       ((uint32_t)(q2 & 0xff) << 16) | ((uint32_t)(q3 & 0xff) << 24);
            }
        }
    }
}

// Quantizes v[0..KP) (KP = k, a power of two >= 4).  packed[j / 4] receives the signed int8 levels,
// little end first; acc[j] += q_j * (norm / levels), the dequantised value.  Returns the norm.
template <int KP>
__device__ __forceinline__ float quantize_bucket(const float (&v)[KP], int levels, uint64_t hnode, int64_t slice,
                                                 uint32_t (&packed)[KP / 4], float (&acc)[KP])
{
    float t[KP / 2];
#pragma unroll
    for (int j = 0; j < KP / 2; ++j) t[j] = __fadd_rn(__fmul_rn(v[j], v[j]), __fmul_rn(v[j + KP / 2], v[j + KP / 2]));
    const float norm = norm_from_first_level<KP / 2>(t);
    quantize_columns<KP>(v, 0, bucket_keys(norm, levels, hnode, slice), packed, acc);
    return norm;
}

}  // namespace quant
}  // namespace gvq
