// Small device helpers shared by the kernels: tile lookup, typed 8-element loads and stores,
// fixed-order block reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "apollo_internal.h"

namespace apollo {

// Debug build (-DAPOLLO_DEBUG): every kernel checks the index range of its global loads and stores against
// the extent of the array before the access; a range that is not inside sets the status word to STATUS_BOUNDS
// and the access is skipped (the kernel goes on and ends normally).  In the release build the macro is `true`.
#ifdef APOLLO_DEBUG
__device__ __forceinline__ bool dbg_in_range(int64_t first, int64_t last, int64_t extent, int32_t* status)
{
    if (first >= 0 && last >= first && last < extent) return true;
    if (status) atomicExch(status, STATUS_BOUNDS);
    return false;
}
#define APOLLO_DBG_RANGE(first, last, extent, status) \
    apollo::dbg_in_range((int64_t)(first), (int64_t)(last), (int64_t)(extent), (status))
#else
#define APOLLO_DBG_RANGE(first, last, extent, status) true
#endif

// prefix[i] = first tile of matrix i, prefix[n_mat] = total.  Returns the matrix that owns
// `tile` (the last i with prefix[i] <= tile; matrices without tiles are skipped).
__device__ __forceinline__ int find_matrix(const int* __restrict__ prefix, int n_mat, int tile)
{
    int lo = 0, hi = n_mat;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(prefix + mid) <= tile) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16)
{
    return __uint_as_float(bits16 << 16);
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& raw, float (&v)[8])
{
    v[0] = __uint_as_float(raw.x << 16); v[1] = __uint_as_float(raw.x & 0xFFFF0000u);
    v[2] = __uint_as_float(raw.y << 16); v[3] = __uint_as_float(raw.y & 0xFFFF0000u);
    v[4] = __uint_as_float(raw.z << 16); v[5] = __uint_as_float(raw.z & 0xFFFF0000u);
    v[6] = __uint_as_float(raw.w << 16); v[7] = __uint_as_float(raw.w & 0xFFFF0000u);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}

__device__ __forceinline__ float load1(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load1(const __nv_bfloat16* p)
{
    return bf16_bits_to_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)));
}

// Eight consecutive elements starting at a 16-byte aligned address.
__device__ __forceinline__ void load8_aligned(const float* p, float (&v)[8])
{
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8_aligned(const __nv_bfloat16* p, float (&v)[8])
{
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p));
    unpack_bf16x8(raw, v);
}

// The same for data that is read once: streaming loads that do not linger in L1.
__device__ __forceinline__ void load8_stream(const float* p, float (&v)[8])
{
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
    const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8_stream(const __nv_bfloat16* p, float (&v)[8])
{
    const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(p));
    unpack_bf16x8(raw, v);
}

// Eight elements as loaded (16 bytes of bf16 / 32 bytes of fp32), unpacked only when used, so that
// many loads can be in flight per thread without holding eight floats each.
template <typename T> struct Raw8;
template <> struct Raw8<float> { float4 a, b; };
template <> struct Raw8<__nv_bfloat16> { uint4 v; };
__device__ __forceinline__ Raw8<float> load_raw8_stream(const float* p)
{
    Raw8<float> r;
    r.a = __ldcs(reinterpret_cast<const float4*>(p));
    r.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    return r;
}
__device__ __forceinline__ Raw8<__nv_bfloat16> load_raw8_stream(const __nv_bfloat16* p)
{
    Raw8<__nv_bfloat16> r;
    r.v = __ldcs(reinterpret_cast<const uint4*>(p));
    return r;
}
__device__ __forceinline__ void unpack_raw8(const Raw8<float>& r, float (&v)[8])
{
    v[0] = r.a.x; v[1] = r.a.y; v[2] = r.a.z; v[3] = r.a.w; v[4] = r.b.x; v[5] = r.b.y; v[6] = r.b.z; v[7] = r.b.w;
}
__device__ __forceinline__ void unpack_raw8(const Raw8<__nv_bfloat16>& r, float (&v)[8]) { unpack_bf16x8(r.v, v); }

// Up to eight consecutive elements with scalar loads; entries at or past `count` read as 0.
template <typename T>
__device__ __forceinline__ void load8_guarded(const T* p, int count, float (&v)[8])
{
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = e < count ? load1(p + e) : 0.0f;
}

// Moment storage: fp32, or bfloat16 behind the same pointer (rounded to nearest even on store).
__device__ __forceinline__ float state_load(const float* base, int64_t idx, bool bf16)
{
    return bf16 ? bf16_bits_to_float((uint32_t)reinterpret_cast<const unsigned short*>(base)[idx]) : base[idx];
}
__device__ __forceinline__ void state_store(float* base, int64_t idx, float v, bool bf16)
{
    if (bf16) reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(v);
    else base[idx] = v;
}

// Sum of one double per thread over the block, in a fixed order (deterministic).
// `scratch` holds at least 32 doubles; every thread gets the result.
__device__ __forceinline__ double block_sum(double v, double* scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double total = 0.0;
    for (int w = 0; w < warps; ++w) total += scratch[w];
    return total;
}

}  // namespace apollo
