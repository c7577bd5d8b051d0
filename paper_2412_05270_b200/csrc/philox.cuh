// Counter-based generator for the projection matrix P (Algorithm 1, "P_t <- N_seed(0, 1/r)").
//
// Philox4x32-10 (Salmon et al., SC'11) keyed by the 64-bit seed, counter
// (column quad q, row k, matrix index, epoch); the four output words become the four
// standard normals Z[k][4q..4q+3] by two Box-Muller transforms.  P = Z / sqrt(r) with Z
// held in bfloat16; the 1/sqrt(r) factor is applied to R = P G by the consumer.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace apollo {

__device__ __forceinline__ void philox_round(uint32_t& c0, uint32_t& c1, uint32_t& c2, uint32_t& c3,
                                             uint32_t k0, uint32_t k1)
{
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;     // one 32x32->64 multiply each
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        philox_round(c0, c1, c2, c3, k0, k1);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Same function with the ten round keys precomputed (kernel parameters: the additions of the
// key schedule disappear and the keys are read as constant-bank operands).
__device__ __forceinline__ uint4 philox4x32_10_keys(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                    const uint32_t (&rk)[20])
{
#pragma unroll
    for (int round = 0; round < 10; ++round) philox_round(c0, c1, c2, c3, rk[2 * round], rk[2 * round + 1]);
    return make_uint4(c0, c1, c2, c3);
}

// The top 23 bits of a word as a float in [1, 2): 1 + (x >> 9) / 2^23 (one funnel shift).
__device__ __forceinline__ float unit_interval_12(uint32_t x)
{
    return __uint_as_float(__funnelshift_r(x, 0x7Fu, 9));
}

// Box-Muller on two words:  u1 = 1 - (xa >> 9) / 2^23 in (0, 1],
// angle = 2 pi ((xb >> 9) / 2^23 - 1/2) in [-pi, pi);  za = radius cos, zb = radius sin with
// radius = sqrt(-2 ln u1).  Fast version: special-function unit approximations.
__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& za, float& zb)
{
    const float u1 = 2.0f - unit_interval_12(xa);
    const float ang = (unit_interval_12(xb) - 1.5f) * 6.283185307179586f;
    float lg, radius, sn, cs;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(u1));
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(radius) : "f"(lg * -1.3862943611198906f));   // -2 ln 2 log2(u1)
    asm("sin.approx.ftz.f32 %0, %1;" : "=f"(sn) : "f"(ang));
    asm("cos.approx.ftz.f32 %0, %1;" : "=f"(cs) : "f"(ang));
    za = radius * cs;
    zb = radius * sn;
}

// Same transform with the full-precision logarithm, sine and cosine (a few ulp): used where
// the generator is a negligible share of the work and P stays in fp32.
__device__ __forceinline__ void box_muller_precise(uint32_t xa, uint32_t xb, float& za, float& zb)
{
    const float u1 = 2.0f - unit_interval_12(xa);
    const float turn = unit_interval_12(xb) - 1.5f;   // [-0.5, 0.5)
    const float radius = sqrtf(-2.0f * logf(u1));
    float sn, cs;
    sincospif(2.0f * turn, &sn, &cs);
    za = radius * cs;
    zb = radius * sn;
}

// The four standard normals of quad q in row k (precise transform).
__device__ __forceinline__ float4 normal_quad(uint32_t q, uint32_t k, uint32_t matrix, uint32_t epoch,
                                              uint32_t key0, uint32_t key1)
{
    const uint4 x = philox4x32_10(q, k, matrix, epoch, key0, key1);
    float4 z;
    box_muller_precise(x.x, x.y, z.x, z.y);
    box_muller_precise(x.z, x.w, z.z, z.w);
    return z;
}

// The same quad with the fast transform, for the tensor-core path, which rounds the result
// to bfloat16 anyway.
__device__ __forceinline__ float4 normal_quad_fast(uint32_t q, uint32_t k, uint32_t matrix, uint32_t epoch,
                                                   const uint32_t (&rk)[20])
{
    const uint4 x = philox4x32_10_keys(q, k, matrix, epoch, rk);
    float4 z;
    box_muller(x.x, x.y, z.x, z.y);
    box_muller(x.z, x.w, z.z, z.w);
    return z;
}

__device__ __forceinline__ float round_to_bf16(float z)
{
    return __bfloat162float(__float2bfloat16_rn(z));
}

}  // namespace apollo
