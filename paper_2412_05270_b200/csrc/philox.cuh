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
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
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

// u1 = ((xa >> 8) + 1) / 2^24 in (0, 1];  angle = 2 pi (xb >> 8) / 2^24, taken modulo
// 2 pi into [-pi, pi) (an arithmetic shift of xb) where the fast sine and cosine are
// most accurate.  za = radius cos, zb = radius sin.
__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& za, float& zb)
{
    const float u1 = (float)((xa >> 8) + 1u) * 5.9604644775390625e-8f;
    const float turn = (float)((int32_t)xb >> 8) * 5.9604644775390625e-8f;   // [-0.5, 0.5)
    const float radius = sqrtf(-2.0f * __logf(u1));
    float sn, cs;
    __sincosf(6.283185307179586f * turn, &sn, &cs);
    za = radius * cs;
    zb = radius * sn;
}

// Same transform with the full-precision logarithm, sine and cosine (a few ulp): used where
// the generator is a negligible share of the work and P stays in fp32.
__device__ __forceinline__ void box_muller_precise(uint32_t xa, uint32_t xb, float& za, float& zb)
{
    const float u1 = (float)((xa >> 8) + 1u) * 5.9604644775390625e-8f;
    const float turn = (float)((int32_t)xb >> 8) * 5.9604644775390625e-8f;   // [-0.5, 0.5)
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

// The same quad with the fast transform (special-function unit approximations), for the
// tensor-core path, which rounds the result to bfloat16 anyway.
__device__ __forceinline__ float4 normal_quad_fast(uint32_t q, uint32_t k, uint32_t matrix, uint32_t epoch,
                                                   uint32_t key0, uint32_t key1)
{
    const uint4 x = philox4x32_10(q, k, matrix, epoch, key0, key1);
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
