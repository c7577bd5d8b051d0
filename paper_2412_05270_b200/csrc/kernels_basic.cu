// Kernels of the APOLLO step that do not use the tensor cores:
//   * the generator by itself (test entry points),
//   * the rank-1 streaming projection (APOLLO-Mini),
//   * the CUDA-core projection with the fused moment update (any rank, dtype, pitch),
//   * the per-matrix finalize (scales, Eq. 5; limiter, Eq. 4),
//   * the fused streaming weight update (Algorithm 1, step 4).
// All launches are grouped over the whole parameter list: a tile index is mapped to its
// matrix through a prefix table.
#include "kernels.h"

#include "device_utils.cuh"
#include "philox.cuh"

namespace apollo {

// ----------------------------------------------------------------------------------------
// Generator test kernels
// ----------------------------------------------------------------------------------------
__global__ void philox_draws_kernel(uint32_t key0, uint32_t key1, uint32_t matrix, uint32_t epoch,
                                    int r, int quads, uint32_t* __restrict__ out)
{
    const int64_t total = (int64_t)r * quads;
    for (int64_t at = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; at < total;
         at += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t k = (uint32_t)(at / quads), q = (uint32_t)(at % quads);
        const uint4 x = philox4x32_10(q, k, matrix, epoch, key0, key1);
        reinterpret_cast<uint4*>(out)[at] = x;
    }
}

__global__ void projection_kernel(uint32_t key0, uint32_t key1, uint32_t matrix, uint32_t epoch,
                                  int r, int m, float* __restrict__ out)
{
    const int quads = (m + 3) / 4;
    const int64_t total = (int64_t)r * quads;
    for (int64_t at = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; at < total;
         at += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t k = (uint32_t)(at / quads), q = (uint32_t)(at % quads);
        const float4 z = normal_quad(q, k, matrix, epoch, key0, key1);
        const float zz[4] = { z.x, z.y, z.z, z.w };
        for (int e = 0; e < 4; ++e) {
            const int i = 4 * (int)q + e;
            if (i < m) out[(int64_t)k * m + i] = zz[e];
        }
    }
}

static int blocks_for(int64_t total)
{
    const int64_t b = (total + 255) / 256;
    return (int)(b < 1 ? 1 : (b < 4096 ? b : 4096));
}

void launch_philox_draws(uint32_t key0, uint32_t key1, uint32_t matrix, uint32_t epoch, int r, int m,
                         uint32_t* d_out, cudaStream_t stream)
{
    const int quads = (m + 3) / 4;
    philox_draws_kernel<<<blocks_for((int64_t)r * quads), 256, 0, stream>>>(key0, key1, matrix, epoch, r, quads, d_out);
}

void launch_projection(uint32_t key0, uint32_t key1, uint32_t matrix, uint32_t epoch, int r, int m,
                       float* d_out, cudaStream_t stream)
{
    const int quads = (m + 3) / 4;
    projection_kernel<<<blocks_for((int64_t)r * quads), 256, 0, stream>>>(key0, key1, matrix, epoch, r, m, d_out);
}

// ----------------------------------------------------------------------------------------
// Rank-1 streaming projection (APOLLO-Mini): R[j] = sum_i P[i] Gv[i][j] and the squared
// column norms of G, one read of G.  Output: part[slice][j] = {partial R_j, partial |G_j|^2}.
//   wide  (rows <= cols): a tile is STREAM_ROWS rows x STREAM_COLS columns; slice = row block.
//   tall  (rows  > cols): a tile is STREAM_TALL_ROWS stored rows (= channels), whole rows; one slice.
// ----------------------------------------------------------------------------------------
constexpr int STREAM_THREADS = 256;
constexpr int STREAM_TALL_CHUNK = 2048;   // entries of P staged per pass over a tall tile

template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 3)     // three blocks per SM: at most 85 registers
project_stream_kernel(const MatDesc* __restrict__ descs, const int* __restrict__ prefix, int n_mat,
                      int tile_begin, int tile_end, StepParams sp, int32_t* __restrict__ status)
{
    __shared__ float Ps[STREAM_TALL_CHUNK];
    __shared__ float red[2][8][STREAM_COLS];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int tile = tile_begin + blockIdx.x; tile < tile_end; tile += gridDim.x) {
        const int mat = find_matrix(prefix, n_mat, tile);
        const MatDesc& d = descs[mat];
        const int local = tile - __ldg(prefix + mat);
        const T* __restrict__ G = static_cast<const T*>(d.G);
        const int cols = d.cols;
        const bool vec_ok = (cols % 8) == 0;
        const int64_t g_extent = (int64_t)d.rows * cols;      // (index checks of the debug build)
        (void)g_extent; (void)status;

        if (!d.tall) {
            const int tn = local % d.tiles_n, tk = local / d.tiles_n;
            const int i0 = tk * STREAM_ROWS;
            const int rows_here = min(STREAM_ROWS, d.rows - i0);
            __syncthreads();   // readers of Ps / red from the previous tile are done
            for (int q = tid; q < STREAM_ROWS / 4; q += STREAM_THREADS) {
                float4 z;
                if (d.ext_p) {
                    const float* src = d.ext_p + i0 + 4 * q;
                    const int left = d.m - (i0 + 4 * q);
                    z.x = left > 0 ? __ldg(src) : 0.f; z.y = left > 1 ? __ldg(src + 1) : 0.f;
                    z.z = left > 2 ? __ldg(src + 2) : 0.f; z.w = left > 3 ? __ldg(src + 3) : 0.f;
                } else {
                    z = normal_quad((uint32_t)(i0 / 4 + q), 0u, (uint32_t)d.matrix_id, sp.epoch, sp.key0, sp.key1);
                }
                Ps[4 * q + 0] = z.x; Ps[4 * q + 1] = z.y;
                Ps[4 * q + 2] = z.z; Ps[4 * q + 3] = z.w;
            }
            __syncthreads();
            const int j0 = tn * STREAM_COLS + lane * 8;
            const int count = max(0, min(8, cols - j0));
            float accR[8], accG[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) { accR[e] = 0.0f; accG[e] = 0.0f; }
            if (count > 0) {
                int ii = warp;
                if (vec_ok) {
                    // eight rows per pass: all eight 16-byte loads are issued before the first use
                    for (; ii + 56 < rows_here; ii += 64) {
                        if (!APOLLO_DBG_RANGE((int64_t)(i0 + ii) * cols + j0, (int64_t)(i0 + ii + 56) * cols + j0 + 7, g_extent, status)) continue;
                        Raw8<T> raw[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) raw[u] = load_raw8_stream(G + (int64_t)(i0 + ii + 8 * u) * cols + j0);
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            float g[8];
                            unpack_raw8(raw[u], g);
                            const float p = Ps[ii + 8 * u];
#pragma unroll
                            for (int e = 0; e < 8; ++e) { accR[e] = fmaf(p, g[e], accR[e]); accG[e] = fmaf(g[e], g[e], accG[e]); }
                        }
                    }
                }
                for (; ii < rows_here; ii += 8) {
                    float g[8];
                    const T* src = G + (int64_t)(i0 + ii) * cols + j0;
                    if (!APOLLO_DBG_RANGE(src - G, src - G + count - 1, g_extent, status)) continue;
                    if (vec_ok) load8_aligned(src, g); else load8_guarded(src, count, g);
                    const float p = Ps[ii];
#pragma unroll
                    for (int e = 0; e < 8; ++e) { accR[e] = fmaf(p, g[e], accR[e]); accG[e] = fmaf(g[e], g[e], accG[e]); }
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) { red[0][warp][lane * 8 + e] = accR[e]; red[1][warp][lane * 8 + e] = accG[e]; }
            __syncthreads();
            const int j = tn * STREAM_COLS + tid;
            if (j < cols) {
                float r = 0.0f, g2 = 0.0f;
#pragma unroll
                for (int w = 0; w < 8; ++w) { r += red[0][w][tid]; g2 += red[1][w][tid]; }
                float2* out = reinterpret_cast<float2*>(d.part) + ((int64_t)tk * d.n + j);
                if (APOLLO_DBG_RANGE((int64_t)tk * d.n + j, (int64_t)tk * d.n + j, (int64_t)d.slices * d.n, status))
                    *out = make_float2(r * d.r_scale, g2);
            }
        } else {
            // channels are the stored rows; the contraction runs along the contiguous side
            const int j_base = local * STREAM_TALL_ROWS + warp * 8;
            float accR[8], accG[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) { accR[e] = 0.0f; accG[e] = 0.0f; }
            for (int c0 = 0; c0 < cols; c0 += STREAM_TALL_CHUNK) {
                __syncthreads();
                for (int q = tid; q < STREAM_TALL_CHUNK / 4; q += STREAM_THREADS) {
                    float4 z;
                    if (d.ext_p) {
                        const float* src = d.ext_p + c0 + 4 * q;
                        const int left = d.m - (c0 + 4 * q);
                        z.x = left > 0 ? __ldg(src) : 0.f; z.y = left > 1 ? __ldg(src + 1) : 0.f;
                        z.z = left > 2 ? __ldg(src + 2) : 0.f; z.w = left > 3 ? __ldg(src + 3) : 0.f;
                    } else {
                        z = normal_quad((uint32_t)(c0 / 4 + q), 0u, (uint32_t)d.matrix_id, sp.epoch, sp.key0, sp.key1);
                    }
                    Ps[4 * q + 0] = z.x; Ps[4 * q + 1] = z.y;
                    Ps[4 * q + 2] = z.z; Ps[4 * q + 3] = z.w;
                }
                __syncthreads();
                const int chunk = min(STREAM_TALL_CHUNK, cols - c0);
                const int rows_left = d.rows - j_base;     // rows of this warp that exist (<= 0: none)
                for (int x = lane * 8; x < chunk; x += 256) {
                    const int count = min(8, chunk - x);
                    float p[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) p[e] = Ps[x + e];   // entries past `chunk` meet zero-filled g
                    if (vec_ok && rows_left >= 8) {
                        if (!APOLLO_DBG_RANGE((int64_t)j_base * cols + c0 + x, (int64_t)(j_base + 7) * cols + c0 + x + 7, g_extent, status)) continue;
                        // all eight 16-byte loads of the warp's rows are issued before the first use
                        Raw8<T> raw[8];
#pragma unroll
                        for (int rr = 0; rr < 8; ++rr) raw[rr] = load_raw8_stream(G + (int64_t)(j_base + rr) * cols + c0 + x);
#pragma unroll
                        for (int rr = 0; rr < 8; ++rr) {
                            float g[8];
                            unpack_raw8(raw[rr], g);
#pragma unroll
                            for (int e = 0; e < 8; ++e) { accR[rr] = fmaf(p[e], g[e], accR[rr]); accG[rr] = fmaf(g[e], g[e], accG[rr]); }
                        }
                        continue;
                    }
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        if (rr < rows_left) {
                            float g[8];
                            const T* src = G + (int64_t)(j_base + rr) * cols + c0 + x;
                            if (!APOLLO_DBG_RANGE(src - G, src - G + count - 1, g_extent, status)) continue;
                            if (vec_ok) load8_aligned(src, g); else load8_guarded(src, count, g);
#pragma unroll
                            for (int e = 0; e < 8; ++e) { accR[rr] = fmaf(p[e], g[e], accR[rr]); accG[rr] = fmaf(g[e], g[e], accG[rr]); }
                        }
                    }
                }
            }
#pragma unroll
            for (int rr = 0; rr < 8; ++rr) {
                float r = accR[rr], g2 = accG[rr];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    r += __shfl_xor_sync(0xFFFFFFFFu, r, off);
                    g2 += __shfl_xor_sync(0xFFFFFFFFu, g2, off);
                }
                const int j = j_base + rr;
                if (lane == 0 && j < d.rows && APOLLO_DBG_RANGE(j, j, (int64_t)d.slices * d.n, status))
                    reinterpret_cast<float2*>(d.part)[j] = make_float2(r * d.r_scale, g2);
            }
        }
    }
}

// ----------------------------------------------------------------------------------------
// CUDA-core projection with fused epilogue.  A tile is SIMT_BR rows of R x SIMT_BN channels;
// it walks the whole projected side in chunks of SIMT_BK, generating the P chunk into
// shared memory, then updates M and V for its tile and emits per-channel partial sums
//   part[row block][j] = { sum_k R~_kj^2, sum_k R_kj^2 }   and, from row block 0,
//   g2[j] = |G_j|^2.
// ----------------------------------------------------------------------------------------
constexpr int SIMT_THREADS = 256;

template <typename T>
__global__ void __launch_bounds__(SIMT_THREADS)
project_simt_kernel(const MatDesc* __restrict__ descs, const int* __restrict__ prefix, int n_mat,
                    int tile_begin, int tile_end, StepParams sp, int32_t* __restrict__ status)
{
    __shared__ float Ps[SIMT_BK][SIMT_BR + 1];     // [kk][row of R]
    __shared__ float Gs[SIMT_BK][SIMT_BN + 1];     // [kk][channel]
    __shared__ float red[2][16][SIMT_BN];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;       // tx: 4 channels each, ty: 4 rows of R each
    for (int tile = tile_begin + blockIdx.x; tile < tile_end; tile += gridDim.x) {
        const int mat = find_matrix(prefix, n_mat, tile);
        const MatDesc& d = descs[mat];
        const int local = tile - __ldg(prefix + mat);
        const int tn = local % d.tiles_n, tr = local / d.tiles_n;
        const int j0 = tn * SIMT_BN, k0 = tr * SIMT_BR;
        const T* __restrict__ G = static_cast<const T*>(d.G);
        const int cols = d.cols, m = d.m, n = d.n, r = sp.rank;
        const float r_scale = d.r_scale;
        const float* __restrict__ ext_p = d.ext_p;
        const int64_t g_extent = (int64_t)d.rows * cols, state_extent = state_elements(n, r, false);   // (debug build)
        (void)g_extent; (void)state_extent; (void)status;

        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;
        float g2 = 0.0f;   // thread tid < SIMT_BN of row block 0 owns channel j0 + tid

        for (int i0 = 0; i0 < m; i0 += SIMT_BK) {
            __syncthreads();
            // P chunk: SIMT_BR rows x SIMT_BK entries = 8 quads per row
            for (int at = tid; at < SIMT_BR * (SIMT_BK / 4); at += SIMT_THREADS) {
                const int row = at / (SIMT_BK / 4), q = at % (SIMT_BK / 4);
                float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                if (k0 + row < r) {
                    if (ext_p) {
                        const float* src = ext_p + (int64_t)(k0 + row) * m + i0 + 4 * q;
                        const int left = m - (i0 + 4 * q);
                        z.x = left > 0 ? __ldg(src) : 0.f; z.y = left > 1 ? __ldg(src + 1) : 0.f;
                        z.z = left > 2 ? __ldg(src + 2) : 0.f; z.w = left > 3 ? __ldg(src + 3) : 0.f;
                    } else {
                        z = normal_quad((uint32_t)(i0 / 4 + q), (uint32_t)(k0 + row), (uint32_t)d.matrix_id, sp.epoch,
                                        sp.key0, sp.key1);
                    }
                }
                if (sizeof(T) == 2) {   // bf16 gradients: P has the precision of the GEMM operands
                    z.x = round_to_bf16(z.x); z.y = round_to_bf16(z.y); z.z = round_to_bf16(z.z); z.w = round_to_bf16(z.w);
                }
                Ps[4 * q + 0][row] = z.x; Ps[4 * q + 1][row] = z.y;
                Ps[4 * q + 2][row] = z.z; Ps[4 * q + 3][row] = z.w;
            }
            // G chunk: Gs[kk][jj] = Gv[i0+kk][j0+jj], zero outside the matrix
            if (!d.tall) {
                for (int at = tid; at < SIMT_BK * SIMT_BN; at += SIMT_THREADS) {
                    const int kk = at / SIMT_BN, jj = at % SIMT_BN;
                    const int i = i0 + kk, j = j0 + jj;
                    Gs[kk][jj] = (i < m && j < n && APOLLO_DBG_RANGE((int64_t)i * cols + j, (int64_t)i * cols + j, g_extent, status))
                                     ? load1(G + (int64_t)i * cols + j) : 0.0f;
                }
            } else {
                for (int at = tid; at < SIMT_BK * SIMT_BN; at += SIMT_THREADS) {
                    const int jj = at / SIMT_BK, kk = at % SIMT_BK;
                    const int i = i0 + kk, j = j0 + jj;
                    Gs[kk][jj] = (i < m && j < n && APOLLO_DBG_RANGE((int64_t)j * cols + i, (int64_t)j * cols + i, g_extent, status))
                                     ? load1(G + (int64_t)j * cols + i) : 0.0f;
                }
            }
            __syncthreads();
#pragma unroll 8
            for (int kk = 0; kk < SIMT_BK; ++kk) {
                float a[4], b[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) { a[x] = Ps[kk][ty * 4 + x]; b[x] = Gs[kk][tx * 4 + x]; }
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
            }
            if (tr == 0 && tid < SIMT_BN) {
#pragma unroll 8
                for (int kk = 0; kk < SIMT_BK; ++kk) g2 = fmaf(Gs[kk][tid], Gs[kk][tid], g2);
            }
        }

        // epilogue: moments and per-channel partial sums
        float num[4] = { 0.f, 0.f, 0.f, 0.f }, den[4] = { 0.f, 0.f, 0.f, 0.f };
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const int k = k0 + ty * 4 + x;
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const int j = j0 + tx * 4 + y;
                if (k < r && j < n && APOLLO_DBG_RANGE((int64_t)k * d.ns + j, (int64_t)k * d.ns + j, state_extent, status)) {
                    const float rv = acc[x][y] * r_scale;
                    const int64_t at = (int64_t)k * d.ns + j;
                    const bool sb = sp.state_bf16 != 0;
                    const float mv = sp.beta1 * state_load(d.M, at, sb) + (1.0f - sp.beta1) * rv;
                    const float vv = sp.beta2 * state_load(d.V, at, sb) + (1.0f - sp.beta2) * rv * rv;
                    state_store(d.M, at, mv, sb); state_store(d.V, at, vv, sb);
                    const float rt = (mv * sp.inv_bc1) / (sqrtf(vv * sp.inv_bc2) + sp.eps);
                    num[y] = fmaf(rt, rt, num[y]);
                    den[y] = fmaf(rv, rv, den[y]);
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int y = 0; y < 4; ++y) { red[0][ty][tx * 4 + y] = num[y]; red[1][ty][tx * 4 + y] = den[y]; }
        __syncthreads();
        if (tid < SIMT_BN && j0 + tid < n &&
            APOLLO_DBG_RANGE((int64_t)tr * n + j0 + tid, (int64_t)tr * n + j0 + tid, (int64_t)d.slices * n, status)) {
            float a = 0.f, b = 0.f;
#pragma unroll
            for (int w = 0; w < 16; ++w) { a += red[0][w][tid]; b += red[1][w][tid]; }
            reinterpret_cast<float2*>(d.part)[(int64_t)tr * n + j0 + tid] = make_float2(a, b);
            if (tr == 0) d.g2[j0 + tid] = g2;
        }
    }
}

// ----------------------------------------------------------------------------------------
// Finalize: one block per matrix.  Sums the partials in a fixed order, (for the streaming
// path) updates the rank-1 moments, forms the scales (Eq. 5 / tensor-wise) and applies the
// norm-growth limiter (Eq. 4) to |G diag(s)|_F = sqrt(sum_j s_j^2 |G_j|^2).
// ----------------------------------------------------------------------------------------
constexpr int FINALIZE_THREADS = 1024;

__global__ void __launch_bounds__(FINALIZE_THREADS)
finalize_kernel(const MatDesc* __restrict__ descs, int first, StepParams sp, int32_t* __restrict__ status)
{
    __shared__ double scratch[32];
    if (status && *status != STATUS_OK) return;      // the projection did not complete: leave s, prev and scal alone
    const MatDesc& d = descs[first + blockIdx.x];
    const int n = d.n;
    const bool tensor_mode = sp.mode == 1;
    double sum_num = 0.0, sum_den = 0.0, sum_g2 = 0.0, sum_sq = 0.0;

    for (int j = threadIdx.x; j < n; j += blockDim.x) {
        float num = 0.f, den = 0.f, g2 = 0.f;
        if (!APOLLO_DBG_RANGE(j, (int64_t)(d.slices - 1) * n + j, (int64_t)d.slices * n, status)) continue;
        if (d.path == PATH_STREAM) {
            float r = 0.f;
            for (int sl = 0; sl < d.slices; ++sl) {
                const float2 p = reinterpret_cast<const float2*>(d.part)[(int64_t)sl * n + j];
                r += p.x; g2 += p.y;
            }
            const bool sb = sp.state_bf16 != 0;
            const float mv = sp.beta1 * state_load(d.M, j, sb) + (1.0f - sp.beta1) * r;
            const float vv = sp.beta2 * state_load(d.V, j, sb) + (1.0f - sp.beta2) * r * r;
            state_store(d.M, j, mv, sb); state_store(d.V, j, vv, sb);
            const float rt = (mv * sp.inv_bc1) / (sqrtf(vv * sp.inv_bc2) + sp.eps);
            num = rt * rt; den = r * r;
        } else {
            for (int sl = 0; sl < d.slices; ++sl) {
                const float2 p = reinterpret_cast<const float2*>(d.part)[(int64_t)sl * n + j];
                num += p.x; den += p.y;
            }
            for (int sl = 0; sl < d.g2_slices; ++sl) g2 += d.g2[(int64_t)sl * n + j];
        }
        if (tensor_mode) {
            sum_num += (double)num; sum_den += (double)den; sum_g2 += (double)g2;
        } else {
            const float s = den > 0.f ? sqrtf(num) / sqrtf(den) : 0.f;
            d.s[j] = s;
            sum_sq += (double)s * (double)s * (double)g2;
        }
    }
    float s_tensor = 0.f;
    if (tensor_mode) {
        const double tn = block_sum(sum_num, scratch);
        const double td = block_sum(sum_den, scratch);
        const double tg = block_sum(sum_g2, scratch);
        s_tensor = td > 0.0 ? (float)(sqrt(tn) / sqrt(td)) : 0.f;
        for (int j = threadIdx.x; j < n; j += blockDim.x) d.s[j] = s_tensor;
        sum_sq = (double)s_tensor * (double)s_tensor * tg;
    } else {
        sum_sq = block_sum(sum_sq, scratch);
    }
    if (threadIdx.x == 0) {
        const float raw = (float)sqrt(sum_sq);
        const float prev = *d.prev;
        float c = 1.0f, norm = raw;
        if (sp.gamma > 0.f && prev > 0.f && raw > sp.gamma * prev) {
            c = sp.gamma * prev / raw;
            norm = sp.gamma * prev;
        }
        *d.prev = norm;
        d.scal[0] = norm; d.scal[1] = c; d.scal[2] = raw; d.scal[3] = s_tensor;
    }
}

// ----------------------------------------------------------------------------------------
// Fused update (Algorithm 1, step 4): W <- W - lr (alpha c s_j G + wd W), one streaming
// pass over the flat rows*cols array in 16-byte vectors.  The scale index is the column
// (wide) or the stored row (tall).
// ----------------------------------------------------------------------------------------
constexpr int UPDATE_THREADS = UPDATE_BLOCK;

__device__ __forceinline__ void store8(float* p, const float (&v)[8])
{
    __stcs(reinterpret_cast<float4*>(p), make_float4(v[0], v[1], v[2], v[3]));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(v[4], v[5], v[6], v[7]));
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8])
{
    uint4 raw;
    raw.x = pack_bf16x2(v[0], v[1]); raw.y = pack_bf16x2(v[2], v[3]);
    raw.z = pack_bf16x2(v[4], v[5]); raw.w = pack_bf16x2(v[6], v[7]);
    __stcs(reinterpret_cast<uint4*>(p), raw);
}
__device__ __forceinline__ void store1(float* p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(UPDATE_THREADS)
update_kernel(const MatDesc* __restrict__ descs, const int* __restrict__ prefix, int n_mat,
              int tile_begin, int tile_end, StepParams sp, int32_t* __restrict__ status)
{
    if (status && *status != STATUS_OK) return;      // the projection did not complete: leave W alone
    for (int tile = tile_begin + blockIdx.x; tile < tile_end; tile += gridDim.x) {
        const int mat = find_matrix(prefix, n_mat, tile);
        const MatDesc& d = descs[mat];
        const int local = tile - __ldg(prefix + mat);
        T* __restrict__ W = static_cast<T*>(d.W);
        const T* __restrict__ G = static_cast<const T*>(d.G);
        const float* __restrict__ s = d.s;
        const uint32_t cols = (uint32_t)d.cols;
        const int64_t total = (int64_t)d.rows * d.cols;
        const int64_t e0 = (int64_t)local * UPDATE_TILE;
        const int64_t row0 = e0 / cols;
        const uint32_t col0 = (uint32_t)(e0 - row0 * cols);
        const float step = sp.lr * sp.alpha * d.scal[1];
        const float decay = sp.lr * sp.wd;
        const bool tall = d.tall != 0;

        if (d.upd_chunks > 0) {
            // 2-D tile: `groups` groups of UPDATE_ROWS rows x one column chunk; this thread owns eight
            // columns of the chunk in one of the groups
            const int chunks = d.upd_chunks, cw = d.upd_width, tpr = cw >> 3;
            // over super-rows of 8 stored rows when the stored rows are not whole vectors
            const bool sup = d.upd_super != 0;
            const uint32_t ecols = sup ? cols * 8u : cols;
            const int erows = sup ? d.rows >> 3 : d.rows;
            const int rb = local / chunks, ct = local - rb * chunks;
            const int grp = threadIdx.x / tpr, lt = threadIdx.x - grp * tpr;
            const uint32_t c = (uint32_t)ct * (uint32_t)cw + (uint32_t)lt * 8u;
            const int r0 = (rb * d.upd_groups + grp) * UPDATE_ROWS;
            if (grp >= d.upd_groups || c >= ecols || r0 >= erows) continue;
            const int nr = min(UPDATE_ROWS, erows - r0);
            if (!APOLLO_DBG_RANGE((int64_t)r0 * ecols + c, (int64_t)(r0 + nr - 1) * ecols + c + 7, total, status)) continue;
            if (!sup && !APOLLO_DBG_RANGE(tall ? r0 : (int)c, tall ? r0 + nr - 1 : (int)c + 7, d.n, status)) continue;
            float sa[8];                               // step x scale of this thread's columns (wide)
            if (sup) {
                uint32_t col = c % cols;               // the same in every super-row
#pragma unroll
                for (int x = 0; x < 8; ++x) { sa[x] = step * __ldg(s + col); if (++col == cols) col = 0; }
            } else if (!tall) {
                const float4 s0 = __ldg(reinterpret_cast<const float4*>(s + c));
                const float4 s1 = __ldg(reinterpret_cast<const float4*>(s + c + 4));
                sa[0] = step * s0.x; sa[1] = step * s0.y; sa[2] = step * s0.z; sa[3] = step * s0.w;
                sa[4] = step * s1.x; sa[5] = step * s1.y; sa[6] = step * s1.z; sa[7] = step * s1.w;
            }
            const int64_t base = (int64_t)r0 * ecols + c;
            float* const dWp = d.dW;
            auto finish = [&](int r, const float (&g)[8], const float (&w)[8]) {
                const int64_t e = base + (int64_t)r * ecols;
                float dw[8], wn[8];
                if (tall) {
                    const float sv = step * __ldg(s + r0 + r);
#pragma unroll
                    for (int x = 0; x < 8; ++x) dw[x] = -__fmaf_rn(sv, g[x], __fmul_rn(decay, w[x]));
                } else {
#pragma unroll
                    for (int x = 0; x < 8; ++x) dw[x] = -__fmaf_rn(sa[x], g[x], __fmul_rn(decay, w[x]));
                }
#pragma unroll
                for (int x = 0; x < 8; ++x) wn[x] = __fadd_rn(w[x], dw[x]);
                store8(W + e, wn);
                if (dWp) store8(dWp + e, dw);
            };
            if (nr == UPDATE_ROWS) {
                // whole tile: the loads of four rows are issued before the first use
#pragma unroll
                for (int rq = 0; rq < UPDATE_ROWS; rq += 4) {
                    Raw8<T> gr[4], wr[4];
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        gr[v] = load_raw8_stream(G + base + (int64_t)(rq + v) * ecols);
                        wr[v] = load_raw8_stream(W + base + (int64_t)(rq + v) * ecols);
                    }
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        float g[8], w[8];
                        unpack_raw8(gr[v], g); unpack_raw8(wr[v], w);
                        finish(rq + v, g, w);
                    }
                }
            } else {
                for (int r = 0; r < nr; ++r) {
                    float g[8], w[8];
                    load8_aligned(G + base + (int64_t)r * ecols, g);
                    load8_aligned(W + base + (int64_t)r * ecols, w);
                    finish(r, g, w);
                }
            }
            continue;
        }

        constexpr int VECS = UPDATE_TILE / (UPDATE_THREADS * 8);   // vectors per thread per tile
        constexpr int BATCH = 4;                                   // vectors whose loads are issued together
        if (!APOLLO_DBG_RANGE(e0, e0, total, status)) continue;
        if (e0 + UPDATE_TILE <= total) {
            // whole tile inside the matrix: every vector is full; issue a batch of loads first
#pragma unroll 1
            for (int b0 = 0; b0 < VECS; b0 += BATCH) {
                float g[BATCH][8], w[BATCH][8];
#pragma unroll
                for (int v = 0; v < BATCH; ++v) {
                    const int64_t e = e0 + (uint32_t)((b0 + v) * UPDATE_THREADS + threadIdx.x) * 8u;
                    load8_stream(G + e, g[v]);
                    load8_stream(W + e, w[v]);
                }
#pragma unroll
                for (int v = 0; v < BATCH; ++v) {
                    const uint32_t off = (uint32_t)((b0 + v) * UPDATE_THREADS + threadIdx.x) * 8u;
                    const int64_t e = e0 + off;
                    const uint32_t cc = col0 + off;
                    const uint32_t radd = cc / cols;
                    uint32_t col = cc - radd * cols;
                    uint32_t row = (uint32_t)row0 + radd;
                    float a[8];
                    if (tall) {
                        if (col + 8 <= cols) {
                            const float sv = __ldg(s + row);
#pragma unroll
                            for (int x = 0; x < 8; ++x) a[x] = sv;
                        } else {
#pragma unroll
                            for (int x = 0; x < 8; ++x) { a[x] = __ldg(s + row); if (++col >= cols) { col = 0; ++row; } }
                        }
                    } else if (col + 8 <= cols && (col & 3) == 0) {
                        const float4 s0 = __ldg(reinterpret_cast<const float4*>(s + col));
                        const float4 s1 = __ldg(reinterpret_cast<const float4*>(s + col + 4));
                        a[0] = s0.x; a[1] = s0.y; a[2] = s0.z; a[3] = s0.w; a[4] = s1.x; a[5] = s1.y; a[6] = s1.z; a[7] = s1.w;
                    } else {
#pragma unroll
                        for (int x = 0; x < 8; ++x) { a[x] = __ldg(s + col); if (++col >= cols) col = 0; }
                    }
                    float dw[8], wn[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        dw[x] = -__fmaf_rn(step * a[x], g[v][x], __fmul_rn(decay, w[v][x]));
                        wn[x] = __fadd_rn(w[v][x], dw[x]);
                    }
                    store8(W + e, wn);
                    if (d.dW) store8(d.dW + e, dw);
                }
            }
        } else {
            // last tile of a matrix: guarded vectors and a scalar tail
            for (int it = 0; it < VECS; ++it) {
                const uint32_t off = (uint32_t)(it * UPDATE_THREADS + threadIdx.x) * 8u;
                const int64_t e = e0 + off;
                if (e >= total) break;
                const uint32_t cc = col0 + off;
                const uint32_t radd = cc / cols;
                uint32_t col = cc - radd * cols;
                int64_t row = row0 + radd;
                const int count = (int)min((int64_t)8, total - e);
                float g[8], w[8], a[8];
                if (count == 8) { load8_aligned(G + e, g); load8_aligned(W + e, w); }
                else { load8_guarded(G + e, count, g); load8_guarded(W + e, count, w); }
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    a[x] = x < count ? __ldg(s + (tall ? (uint32_t)row : col)) : 0.f;
                    if (++col >= cols) { col = 0; ++row; }
                }
                float dw[8], wn[8];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    dw[x] = -__fmaf_rn(step * a[x], g[x], __fmul_rn(decay, w[x]));
                    wn[x] = __fadd_rn(w[x], dw[x]);
                }
                if (count == 8) {
                    store8(W + e, wn);
                    if (d.dW) store8(d.dW + e, dw);
                } else {
                    for (int x = 0; x < count; ++x) {
                        store1(W + e + x, wn[x]);
                        if (d.dW) d.dW[e + x] = dw[x];
                    }
                }
            }
        }
    }
}

__global__ void state_copy_kernel(void* __restrict__ lib, void* __restrict__ dense, int rank, int rank_layout, int n, int ns,
                                  bool tiled, int lib_esz, int dense_esz, bool to_dense)
{
    const int64_t count = (int64_t)rank * n;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
        const int k = (int)(i / n), j = (int)(i - (int64_t)k * n);
        const int64_t at = state_at(tiled, ns, rank_layout, k, j);
        if (to_dense) {
            if (lib_esz == 4) static_cast<float*>(dense)[i] = static_cast<const float*>(lib)[at];
            else if (dense_esz == 4) static_cast<float*>(dense)[i] = bf16_bits_to_float((uint32_t)static_cast<const unsigned short*>(lib)[at]);
            else static_cast<unsigned short*>(dense)[i] = static_cast<const unsigned short*>(lib)[at];
        } else {
            if (lib_esz == 4) static_cast<float*>(lib)[at] = static_cast<const float*>(dense)[i];
            else static_cast<unsigned short*>(lib)[at] = static_cast<const unsigned short*>(dense)[i];
        }
    }
}

void launch_state_copy(void* d_lib, void* d_dense, int rank, int rank_layout, int n, int ns, bool tiled, int lib_esz,
                       int dense_esz, bool to_dense, cudaStream_t stream)
{
    const int64_t count = (int64_t)rank * n;
    if (count == 0) return;
    state_copy_kernel<<<blocks_for(count), 256, 0, stream>>>(d_lib, d_dense, rank, rank_layout, n, ns, tiled, lib_esz, dense_esz, to_dense);
}

// ----------------------------------------------------------------------------------------
// Launch wrappers
// ----------------------------------------------------------------------------------------
static int grid_for(int total_tiles, int per_sm, int sm_count)
{
    const int cap = per_sm * sm_count;
    return total_tiles < cap ? total_tiles : cap;
}

void launch_project_stream(int dtype, const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                           const StepParams& sp, int sm_count, int32_t* d_status, cudaStream_t stream)
{
    const int total_tiles = tile_end - tile_begin;
    if (total_tiles <= 0) return;
    const int grid = grid_for(total_tiles, 6, sm_count);
    if (dtype == 0)
        project_stream_kernel<float><<<grid, STREAM_THREADS, 0, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, d_status);
    else
        project_stream_kernel<__nv_bfloat16><<<grid, STREAM_THREADS, 0, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, d_status);
}

void launch_project_simt(int dtype, const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                         const StepParams& sp, int sm_count, int32_t* d_status, cudaStream_t stream)
{
    const int total_tiles = tile_end - tile_begin;
    if (total_tiles <= 0) return;
    const int grid = grid_for(total_tiles, 4, sm_count);
    if (dtype == 0)
        project_simt_kernel<float><<<grid, SIMT_THREADS, 0, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, d_status);
    else
        project_simt_kernel<__nv_bfloat16><<<grid, SIMT_THREADS, 0, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, d_status);
}

void launch_finalize(const MatDesc* d_descs, int first, int count, const StepParams& sp, int32_t* d_status,
                     cudaStream_t stream)
{
    if (count <= 0) return;
    finalize_kernel<<<count, FINALIZE_THREADS, 0, stream>>>(d_descs, first, sp, d_status);
}

void launch_update(int dtype, const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                   const StepParams& sp, int sm_count, int32_t* d_status, cudaStream_t stream)
{
    const int total_tiles = tile_end - tile_begin;
    if (total_tiles <= 0) return;
    const int grid = grid_for(total_tiles, 8, sm_count);
    if (dtype == 0)
        update_kernel<float><<<grid, UPDATE_THREADS, 0, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, d_status);
    else
        update_kernel<__nv_bfloat16><<<grid, UPDATE_THREADS, 0, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, d_status);
}

}  // namespace apollo
