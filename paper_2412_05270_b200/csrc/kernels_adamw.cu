// Fused AdamW over a list of tensors (the parameters APOLLO does not project: embeddings,
// norms, output head).  Eq. 1 of the paper with decoupled weight decay; bias-corrected moments
// when asked.  One streaming pass: read g, p, m, v; write p, m, v.  Tensors are processed in
// launches of up to ADAMW_CHUNK tensors whose pointers travel as kernel parameters, so no
// workspace is needed.
#include "../../include/apollo.h"

#include <cmath>

#include "device_utils.cuh"

namespace apollo {

constexpr int ADAMW_CHUNK = 32;
constexpr int ADAMW_TILE = 8192;      // elements per tile
constexpr int ADAMW_THREADS = 256;

struct AdamwArgs {
    void* p[ADAMW_CHUNK];
    const void* g[ADAMW_CHUNK];
    float* m[ADAMW_CHUNK];
    float* v[ADAMW_CHUNK];
    float* dp[ADAMW_CHUNK];           // optional capture of the update, or nullptr
    long long numel[ADAMW_CHUNK];
    int tile_begin[ADAMW_CHUNK + 1];
    int n;
    float lr, beta1, beta2, eps, wd, inv_c1, inv_c2;
};

__device__ __forceinline__ void st8(float* p, const float (&v)[8])
{
    reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void st8(__nv_bfloat16* p, const float (&v)[8])
{
    uint4 raw;
    raw.x = pack_bf16x2(v[0], v[1]); raw.y = pack_bf16x2(v[2], v[3]);
    raw.z = pack_bf16x2(v[4], v[5]); raw.w = pack_bf16x2(v[6], v[7]);
    *reinterpret_cast<uint4*>(p) = raw;
}
__device__ __forceinline__ void st1(float* p, float v) { *p = v; }
__device__ __forceinline__ void st1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(ADAMW_THREADS)
adamw_kernel(const __grid_constant__ AdamwArgs a)
{
    const int total_tiles = a.tile_begin[a.n];
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        int k = 0;
        while (k + 1 < a.n && a.tile_begin[k + 1] <= tile) ++k;
        T* __restrict__ P = static_cast<T*>(a.p[k]);
        const T* __restrict__ G = static_cast<const T*>(a.g[k]);
        float* __restrict__ M = a.m[k];
        float* __restrict__ V = a.v[k];
        float* __restrict__ DP = a.dp[k];
        const long long numel = a.numel[k];
        const long long e0 = (long long)(tile - a.tile_begin[k]) * ADAMW_TILE;
        if (e0 + ADAMW_TILE <= numel) {
            // whole tile: two vectors per thread and pass, all eight loads issued before the first use
#pragma unroll 1
            for (int it = 0; it < ADAMW_TILE / (ADAMW_THREADS * 8); it += 2) {
                float g[2][8], p[2][8], m[2][8], v[2][8];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const long long e = e0 + (long long)((it + u) * ADAMW_THREADS + threadIdx.x) * 8;
                    load8_stream(G + e, g[u]); load8_stream(P + e, p[u]); load8_stream(M + e, m[u]); load8_stream(V + e, v[u]);
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const long long e = e0 + (long long)((it + u) * ADAMW_THREADS + threadIdx.x) * 8;
                    float d[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        m[u][x] = a.beta1 * m[u][x] + (1.0f - a.beta1) * g[u][x];
                        v[u][x] = a.beta2 * v[u][x] + (1.0f - a.beta2) * g[u][x] * g[u][x];
                        const float upd = (m[u][x] * a.inv_c1) / (sqrtf(v[u][x] * a.inv_c2) + a.eps);
                        d[x] = -__fmul_rn(a.lr, __fmaf_rn(a.wd, p[u][x], upd));
                        p[u][x] = __fadd_rn(p[u][x], d[x]);
                    }
                    st8(P + e, p[u]); st8(M + e, m[u]); st8(V + e, v[u]);
                    if (DP) st8(DP + e, d);
                }
            }
            continue;
        }
        for (int it = 0; it < ADAMW_TILE / (ADAMW_THREADS * 8); ++it) {
            const long long e = e0 + (long long)(it * ADAMW_THREADS + threadIdx.x) * 8;
            if (e >= numel) break;
            const int count = (int)min((long long)8, numel - e);
            float g[8], p[8], m[8], v[8], d[8];
            if (count == 8) {
                load8_aligned(G + e, g); load8_aligned(P + e, p); load8_aligned(M + e, m); load8_aligned(V + e, v);
            } else {
                load8_guarded(G + e, count, g); load8_guarded(P + e, count, p);
                load8_guarded(M + e, count, m); load8_guarded(V + e, count, v);
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                m[x] = a.beta1 * m[x] + (1.0f - a.beta1) * g[x];
                v[x] = a.beta2 * v[x] + (1.0f - a.beta2) * g[x] * g[x];
                const float upd = (m[x] * a.inv_c1) / (sqrtf(v[x] * a.inv_c2) + a.eps);
                d[x] = -__fmul_rn(a.lr, __fmaf_rn(a.wd, p[x], upd));
                p[x] = __fadd_rn(p[x], d[x]);
            }
            if (count == 8) {
                st8(P + e, p); st8(M + e, m); st8(V + e, v);
                if (DP) st8(DP + e, d);
            } else {
                for (int x = 0; x < count; ++x) {
                    st1(P + e + x, p[x]); M[e + x] = m[x]; V[e + x] = v[x];
                    if (DP) DP[e + x] = d[x];
                }
            }
        }
    }
}

}  // namespace apollo

using namespace apollo;

extern "C" int apollo_adamw_step(void* const* d_P, const void* const* d_G, float* const* d_M, float* const* d_V,
                                 const int64_t* numel, int32_t n_tensors, int32_t dtype, float lr, float beta1,
                                 float beta2, float eps, float wd, int64_t t, int32_t bias_correction,
                                 float* const* d_dP, void* cuda_stream)
{
    if (!d_P || !d_G || !d_M || !d_V || !numel || n_tensors < 1) return APOLLO_ERR_INVALID_ARG;
    if (dtype != APOLLO_DT_F32 && dtype != APOLLO_DT_BF16) return APOLLO_ERR_INVALID_ARG;
    if (!std::isfinite(lr) || !std::isfinite(wd) || !std::isfinite(eps) || eps < 0.f || t < 0) return APOLLO_ERR_INVALID_ARG;
    if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f)) return APOLLO_ERR_INVALID_ARG;
    for (int i = 0; i < n_tensors; ++i) {
        if (!d_P[i] || !d_G[i] || !d_M[i] || !d_V[i] || numel[i] < 0) return APOLLO_ERR_INVALID_ARG;
        if (numel[i] > (int64_t)INT32_MAX * (ADAMW_TILE / 4)) return APOLLO_ERR_SHAPE;
        if (((uintptr_t)d_P[i] % 16) || ((uintptr_t)d_G[i] % 16) || ((uintptr_t)d_M[i] % 16) || ((uintptr_t)d_V[i] % 16) ||
            (d_dP && d_dP[i] && ((uintptr_t)d_dP[i] % 16)))
            return APOLLO_ERR_ALIGN;
    }
    int device = 0, sms = 0;
    if (cudaGetDevice(&device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        cudaGetLastError();
        return APOLLO_ERR_CUDA;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    float inv_c1 = 1.f, inv_c2 = 1.f;
    if (bias_correction) {
        inv_c1 = (float)(1.0 / (1.0 - std::pow((double)beta1, (double)(t + 1))));
        inv_c2 = (float)(1.0 / (1.0 - std::pow((double)beta2, (double)(t + 1))));
    }
    for (int first = 0; first < n_tensors; first += ADAMW_CHUNK) {
        AdamwArgs a;
        a.n = n_tensors - first < ADAMW_CHUNK ? n_tensors - first : ADAMW_CHUNK;
        a.lr = lr; a.beta1 = beta1; a.beta2 = beta2; a.eps = eps; a.wd = wd; a.inv_c1 = inv_c1; a.inv_c2 = inv_c2;
        long long tiles = 0;
        for (int k = 0; k < ADAMW_CHUNK; ++k) {
            const bool live = k < a.n;
            a.p[k] = live ? d_P[first + k] : nullptr;
            a.g[k] = live ? d_G[first + k] : nullptr;
            a.m[k] = live ? d_M[first + k] : nullptr;
            a.v[k] = live ? d_V[first + k] : nullptr;
            a.dp[k] = live && d_dP ? d_dP[first + k] : nullptr;
            a.numel[k] = live ? numel[first + k] : 0;
            a.tile_begin[k] = (int)tiles;
            if (live) tiles += (numel[first + k] + ADAMW_TILE - 1) / ADAMW_TILE;
            if (tiles > INT32_MAX) return APOLLO_ERR_SHAPE;
        }
        a.tile_begin[ADAMW_CHUNK] = (int)tiles;
        for (int k = a.n; k <= ADAMW_CHUNK; ++k) a.tile_begin[k] = (int)tiles;
        if (tiles == 0) continue;
        const int grid = (int)(tiles < 8LL * sms ? tiles : 8LL * sms);
        if (dtype == APOLLO_DT_F32) adamw_kernel<float><<<grid, ADAMW_THREADS, 0, stream>>>(a);
        else adamw_kernel<__nv_bfloat16><<<grid, ADAMW_THREADS, 0, stream>>>(a);
    }
    return cudaGetLastError() == cudaSuccess ? APOLLO_OK : APOLLO_ERR_CUDA;
}
