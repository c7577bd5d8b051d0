// Tensor-core projection: R = P G on tcgen05 with TMEM accumulators (Algorithm 1, step 1),
// with the moment update and the per-channel norm sums fused into the epilogue (Algorithm 1,
// step 2; Eq. 5).  P tiles come from a scratch in the workspace that L2 keeps: spare warps of the pair
// kernel regenerate every matrix's P from the seed a few matrices ahead of its use (default), or
// generate_p_kernel fills it (once per epoch with APOLLO_FLAG_KEEP_P, else group by group); the ring
// kernel can also generate them straight into shared memory.
//
// Two kernels share this file: project_pair_kernel (default when P is staged; CTA pairs, described
// above its definition) and project_tensor_kernel, the single-CTA ring kernel described here.
//
// Roles of the 14 warps of a ring-kernel CTA (one CTA per SM, persistent over tiles of 256 channels):
//   warp 0      TMA producer: G tiles (and P tiles from the scratch) into a shared-memory ring, 128-byte swizzle
//   warp 1      MMA issuer (one thread) and owner of the 512 TMEM columns
//   warps 2-9   P from the scratch: L2 prefetch of the G lines the producer will ask for next;
//               otherwise generators: Philox -> Box-Muller -> bf16 P tile in the UMMA K-major layout
//   warps 10-13 column norms of G from the landed tiles
//   warps 2-13  epilogue: tcgen05.ld of R, read-modify-write of M and V, partial sums
//
// Operand roles: D[128 channels x r_slice] = A[128 channels x 64] * B[r_slice x 64]^T, so
// a TMEM lane is a channel and the reductions over r are per thread.  A = G tile: K-major
// for a tall matrix (channels are stored rows), MN-major for a wide one.  B = P tile.
//
// Every wait on an mbarrier is bounded.  When one gives up, the CTA sets the status word, stops
// issuing loads and MMAs, leaves the tile loop through a barrier vote, waits (bounded again) for
// the loads and MMAs already in flight, frees its TMEM and returns.
#include "kernels.h"

#include <cuda.h>
#include <cstring>
#include <vector>

#include "../../include/apollo.h"
#include "device_utils.cuh"
#include "philox.cuh"
#include "tc_ptx.cuh"

namespace apollo {

namespace {

constexpr int TC_THREADS = 448;
constexpr int TC_BK = 64;                 // contraction elements per stage (128 bytes of bf16)
constexpr int TC_GEN_THREADS = 256;       // warps 2-9
constexpr int TC_NORM_THREADS = 128;      // warps 10-13
constexpr int TC_EPI_THREADS = 384;       // warps 2-13
constexpr int TC_BLOCK_BYTES = 128 * TC_BK * 2;   // one 128-channel block of a G stage: 16 KiB
constexpr int TC_MISC_BYTES = 256 + 3 * 512 * 8 + 8 * 512 * 4 + 1024;   // barriers, red, g2s, alignment slack
constexpr int TC_MAX_SMEM = 227 * 1024;
constexpr int TC_PREFETCH = 2;             // k-blocks of G asked into L2 ahead of the load that needs them
constexpr uint32_t TC_PACE_CAP = 1u << 12; // polls (100 ns apart) of the prefetchers' pacing wait; expiry is harmless
constexpr uint32_t TC_WAIT_CAP = 1u << 20;   // polls before a wait gives up (normal waits are far below 1 ms)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

// Bytes one matrix's P takes in the scratch: rank rows of round_up(m, 64) bfloat16 standard normals.
// A split matrix (fp32 gradient) keeps the high and the low bfloat16 part of every normal: twice the width.
size_t tensor_path_stage_bytes(int rows, int cols, int rank, bool split)
{
    const int m = rows > cols ? cols : rows;
    return (size_t)rank * (size_t)((m + 63) / 64 * 64) * 2 * (split ? 2 : 1);
}

// The bfloat16 high/low copy of an fp32 gradient: [hi; lo] along the projected side, each part m_pad =
// round_up(m, 64) long (zero beyond m).  Wide: 2 m_pad rows of round_up(cols, 8) elements; tall: rows of 2 m_pad.
size_t tensor_path_split_bytes(int rows, int cols, int* pitch)
{
    const bool tall = rows > cols;
    const int m_pad = ((tall ? cols : rows) + 63) / 64 * 64;
    const int p = tall ? 2 * m_pad : (cols + 7) / 8 * 8;
    if (pitch) *pitch = p;
    return (size_t)(tall ? rows : 2 * m_pad) * (size_t)p * 2;
}

int tensor_path_configure(int rank, uint32_t flags, const apollo_tuning* tuning, TcTiling* out)
{
    static const apollo_tuning defaults = {};
    const apollo_tuning& tu = tuning ? *tuning : defaults;
    TcTiling t = {};
    if (tu.kernel != APOLLO_TC_KERNEL_PAIR && tu.kernel != APOLLO_TC_KERNEL_RING) return APOLLO_ERR_INVALID_ARG;
    if (tu.p_source != APOLLO_P_SCRATCH && tu.p_source != APOLLO_P_SHARED) return APOLLO_ERR_INVALID_ARG;
    if (tu.p_generator < 0 || tu.p_generator > 2) return APOLLO_ERR_INVALID_ARG;
    if (tu.scratch_mb < 0 || tu.scratch_mb > 65536 || tu.realign < 0 || tu.realign > 2) return APOLLO_ERR_INVALID_ARG;
    if (tu.repitch_mb < 0 || tu.repitch_mb > 65536) return APOLLO_ERR_INVALID_ARG;
    if (tu.epi_prefetch < 0 || tu.epi_prefetch > 9) return APOLLO_ERR_INVALID_ARG;
    t.r_slice = rank <= 256 ? rank : rank / 2;
    if (tu.r_slice != 0) {
        if (tu.r_slice < 16 || tu.r_slice > 256 || tu.r_slice % 16 || rank % tu.r_slice) return APOLLO_ERR_INVALID_ARG;
        t.r_slice = tu.r_slice;
    }
    const int fit = 512 / t.r_slice;
    t.nblk = fit >= 4 ? 4 : (fit >= 2 ? 2 : 1);
    if (tu.nblk != 0) {
        if ((tu.nblk != 1 && tu.nblk != 2 && tu.nblk != 4) || tu.nblk * t.r_slice > 512) return APOLLO_ERR_INVALID_ARG;
        t.nblk = tu.nblk;
    }
    t.staged = tu.p_source == APOLLO_P_SCRATCH ? 1 : 0;
    t.keep = t.staged && (flags & APOLLO_FLAG_KEEP_P) ? 1 : 0;
    t.scratch_bytes = (int64_t)(tu.scratch_mb ? tu.scratch_mb : 128) << 20;
    t.repitch_bytes = (int64_t)tu.repitch_mb << 20;      // 0: no limit, every matrix has its own copy (one projection launch)
    t.epi_prefetch = tu.epi_prefetch ? tu.epi_prefetch - 1 : 1;
    t.raw_allowed = tu.realign == 1 ? 1 : 0;      // default: padded copy (5 % faster on the 1B list, at 1.07 GB of workspace)
    // Staged P has two kernels: the pair kernel (default; faster on every list measured) and the single-CTA
    // ring kernel, which is also the one that can generate P in shared memory.
    if (t.staged && tu.kernel == APOLLO_TC_KERNEL_PAIR) {   // (APOLLO_P_SHARED always runs on the ring kernel)
        // pair tile: 256 channels (128 per CTA) x r_slice rows, accumulator double buffered
        t.pair = 1;
        t.nblk = 2;
        t.gen = !t.keep && tu.p_generator != 1 ? (tu.p_generator == 2 ? 2 : 1) : 0;      // 2: also for lists that would fit the scratch
        const int stage = 128 * TC_BK * 2 + (t.r_slice / 2) * 128;
        t.stages = (TC_MAX_SMEM - 1536) / stage;
        if (t.stages > 8) t.stages = 8;
        t.smem_bytes = t.stages * stage + 1536;
        *out = t;
        return APOLLO_OK;
    }
    const int stage = t.nblk * TC_BLOCK_BYTES + t.r_slice * 128;
    t.stages = (TC_MAX_SMEM - TC_MISC_BYTES) / stage;
    if (t.stages > 4) t.stages = 4;
    t.smem_bytes = t.stages * stage + TC_MISC_BYTES;
    *out = t;
    return APOLLO_OK;
}

int tensor_path_padded_rank(int rank)
{
    return rank <= 256 ? (rank + 15) / 16 * 16 : (rank + 31) / 32 * 32;
}

bool tensor_path_supports(int rows, int cols, int rank, int dtype, const TcTiling& tl)
{
    // fp32 gradients go through a bfloat16 high/low split that only the pair kernel with a P scratch reads
    if (dtype != APOLLO_DT_BF16 && !(tl.pair && tl.staged)) return false;
    // any rank from 16 on: the MMA works on the rank rounded up to its granularity, with zero rows of P
    if (rank < 16 || rank > 512) return false;
    (void)rows; (void)cols;   // a row pitch that is not a multiple of 16 bytes goes through a padded copy
    return true;
}

bool tensor_path_raw_ok(int rows, int cols, const TcTiling& tl)
{
    return tl.pair != 0 && tl.raw_allowed != 0 && rows <= cols && (cols % 8) != 0 && (rows % 8) == 0;
}

void tensor_path_enable_raw(TcTiling* tl)
{
    if (!tl->pair || tl->raw) return;
    tl->raw = 1;
    const int stage = RAW_G_BYTES + (tl->r_slice / 2) * 128;
    tl->stages = (TC_MAX_SMEM - 1536) / stage;
    if (tl->stages > 8) tl->stages = 8;
    tl->smem_bytes = tl->stages * stage + 1536;
}

void tensor_path_tiling(int rows, int cols, int rank, const TcTiling& t, int32_t* tiles_n, int32_t* tiles_k,
                        int32_t* slices, int32_t* g2_slices)
{
    const int n = rows > cols ? rows : cols;
    *tiles_n = (n + t.nblk * 128 - 1) / (t.nblk * 128);
    *tiles_k = rank / t.r_slice;
    // partial sums a tile leaves for finalize_kernel: the pair kernel writes one slice per half of its
    // epilogue warps and, for a wide matrix, one slice of squared column norms per norm warp
    *slices = t.pair ? 2 * *tiles_k : *tiles_k;
    *g2_slices = t.pair && rows <= cols ? 4 : 1;
}

int tensor_path_prepare(MatDesc* h_descs, int n_mat, int rank, const TcTiling& tl, void* h_maps)
{
    bool any = false;
    for (int i = 0; i < n_mat; ++i) any |= h_descs[i].path == PATH_TENSOR;
    if (!any) return APOLLO_OK;
    EncodeTiledFn encode = encode_fn();
    if (!encode) return APOLLO_ERR_CUDA;
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    CUtensorMap* maps = static_cast<CUtensorMap*>(h_maps);
    for (int i = 0; i < n_mat; ++i) {
        const MatDesc& d = h_descs[i];
        if (d.path != PATH_TENSOR) continue;
        // dimension 0 is the contiguous one (the stored columns)
        // (a split matrix is read from its high/low copy: the projected side is 2 m_pad long there)
        const cuuint64_t dims[2] = { (cuuint64_t)(d.split && d.tall ? 2 * d.m_pad : d.cols),
                                     (cuuint64_t)(d.split && !d.tall ? 2 * d.m_pad : d.rows) };
        const cuuint64_t strides[1] = { (cuuint64_t)d.g_pitch * 2 };
        // wide: 64 channels x 64 rows of G; tall: 64 contraction elements x 128 channels
        const cuuint32_t box[2] = { 64u, d.tall ? 128u : 64u };
        const cuuint32_t elem[2] = { 1u, 1u };
        CUresult rc;
        if (d.raw) {
            // Rows of `cols` elements with cols % 8 != 0 start on no 16-byte boundary, which a tensor map cannot
            // describe.  Eight stored rows together are whole 16-byte units: the map sees rows/8 "super-rows" of
            // 8 cols elements, and a box is RAW_BOX_W elements of one stored row in each of 8 consecutive
            // super-rows (rows 8 apart start at the same offset within a 16-byte unit).  No swizzle: the pieces
            // are re-aligned in shared memory.
            const cuuint64_t rdims[2] = { (cuuint64_t)d.cols * 8, (cuuint64_t)d.rows / 8 };
            const cuuint64_t rstrides[1] = { (cuuint64_t)d.cols * 16 };
            const cuuint32_t rbox[2] = { (cuuint32_t)RAW_BOX_W, 8u };
            rc = encode(&maps[2 * i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d.G), rdims, rstrides, rbox,
                        elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        } else {
            rc = encode(&maps[2 * i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        d.gpad ? d.gpad : const_cast<void*>(d.G), dims,
                        strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        }
        if (rc != CUDA_SUCCESS) return APOLLO_ERR_CUDA;
        if (tl.staged) {
            // the P slot: rank rows of p_width bf16, loaded as 64 x r_slice boxes (K-major UMMA tiles)
            const cuuint64_t pdims[2] = { (cuuint64_t)d.p_width, (cuuint64_t)rank };
            const cuuint64_t pstrides[1] = { (cuuint64_t)d.p_width * 2 };
            const cuuint32_t pbox[2] = { 64u, (cuuint32_t)(tl.pair ? tl.r_slice / 2 : tl.r_slice) };
            const CUresult rp = encode(&maps[2 * i + 1], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, d.pstage, pdims, pstrides,
                                       pbox, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (rp != CUDA_SUCCESS) return APOLLO_ERR_CUDA;
        }
    }
    return APOLLO_OK;
}

namespace {

// Bounded wait on an mbarrier phase.  On expiry the CTA-wide abort flag and the global
// status word are set; later waits return at once, so the kernel always terminates.
// Bounded wait on an mbarrier phase.  false = this wait, or an earlier one of this CTA, gave up: the
// caller stops issuing work and falls through to the barriers and the drain at the end of the kernel.
// `where` names the wait (role and barrier); the first one of a launch that gives up is kept in the word after
// the status word, for whoever has to find out what stalled.
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                           int where = 0)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;      // the common case costs one poll and no flag read
    if (*abort_flag) return false;
    for (uint32_t i = 0; i < TC_WAIT_CAP; ++i)
        if (ptx::mbar_try_wait(bar, parity)) return true;
    *abort_flag = 1;
    atomicCAS(status + 1, 0, where);
    atomicExch(status, STATUS_TIMEOUT);
    return false;
}

// The same for waits that have slack (an epilogue waiting for its accumulator): sleeps between polls,
// which costs nothing there and saves issue slots, i.e. power, on a board that runs at its power cap.
__device__ __forceinline__ bool wait_phase_idle(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                                int where = 0)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    for (uint32_t i = 0; i < TC_WAIT_CAP; ++i) {
        __nanosleep(200);
        if (ptx::mbar_try_wait(bar, parity)) return true;
    }
    *abort_flag = 1;
    atomicCAS(status + 1, 0, where);
    atomicExch(status, STATUS_TIMEOUT);
    return false;
}

// Bounded wait that neither reads nor sets the abort flag: lets copies and MMAs that are already in
// flight finish before the CTA gives up its shared memory and TMEM.
__device__ __forceinline__ void drain_phase(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < TC_WAIT_CAP; ++i)
        if (ptx::mbar_try_wait(bar, parity)) return;
}

// Counters in global memory that CTAs of one launch signal each other through (P generated by spare warps).
__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(uint32_t* p, uint32_t v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until *counter >= target.  All CTAs of the launch are resident (the grid is sized by the
// occupancy query), so the writers run; the bound covers the case that one of them gave up.  A set status
// word ends the wait at once.  false = gave up (abort flag and status word are set).
__device__ __forceinline__ bool wait_counter(const uint32_t* counter, uint32_t target, volatile int* abort_flag,
                                             int32_t* status, int where = 0)
{
    if (ld_acquire_gpu(counter) >= target) return true;
    if (*abort_flag) return false;
    for (uint32_t i = 0; i < TC_WAIT_CAP; ++i) {
        __nanosleep(256);
        if (ld_acquire_gpu(counter) >= target) return true;
        if ((i & 63u) == 63u && *reinterpret_cast<volatile int32_t*>(status) != STATUS_OK) break;
    }
    *abort_flag = 1;
    atomicCAS(status + 1, 0, where);
    atomicExch(status, STATUS_TIMEOUT);
    return false;
}

// Eight standard normals of row `row`, columns 8 ch .. 8 ch + 7 of a matrix's P as bfloat16 (one 16-byte
// store of the scratch), from the generator or from a projection supplied by the caller.
// SPLIT (fp32 gradients): a row of the slot is [P_hi | P_lo], each half_vpr vectors long: the normals in fp32
// (the precise transform), their bfloat16 rounding and the bfloat16 rounding of what the first rounding left.
template <bool SPLIT>
__device__ __forceinline__ uint4 p_vector(const float* __restrict__ ext_p, int m, int row, int ch, uint32_t matrix_id,
                                          const StepParams& sp, int half_vpr = 0)
{
    uint4 v;
    // rows from `rank` on pad a rank that is not a multiple of 16: zero (selected at the end, without a branch, so that
    // the Philox chains of two calls still interleave)
    const bool pad_row = row >= sp.rank;
    if (SPLIT) {
        const bool low = ch >= half_vpr;
        const int c = low ? ch - half_vpr : ch;
        float z[8];
        if (ext_p) {
#pragma unroll
            for (int e = 0; e < 8; ++e) z[e] = 8 * c + e < m ? __ldg(ext_p + (int64_t)row * m + 8 * c + e) : 0.f;
        } else {
            const float4 a0 = normal_quad((uint32_t)(2 * c), (uint32_t)row, matrix_id, sp.epoch, sp.key0, sp.key1);
            const float4 a1 = normal_quad((uint32_t)(2 * c + 1), (uint32_t)row, matrix_id, sp.epoch, sp.key0, sp.key1);
            z[0] = a0.x; z[1] = a0.y; z[2] = a0.z; z[3] = a0.w; z[4] = a1.x; z[5] = a1.y; z[6] = a1.z; z[7] = a1.w;
        }
        if (low) {
#pragma unroll
            for (int e = 0; e < 8; ++e) z[e] -= round_to_bf16(z[e]);
        }
        v.x = pack_bf16x2(z[0], z[1]); v.y = pack_bf16x2(z[2], z[3]);
        v.z = pack_bf16x2(z[4], z[5]); v.w = pack_bf16x2(z[6], z[7]);
        return pad_row ? make_uint4(0u, 0u, 0u, 0u) : v;
    }
    if (ext_p) {
        float z[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = 8 * ch + e < m ? __ldg(ext_p + (int64_t)row * m + 8 * ch + e) : 0.f;
        v.x = pack_bf16x2(z[0], z[1]); v.y = pack_bf16x2(z[2], z[3]);
        v.z = pack_bf16x2(z[4], z[5]); v.w = pack_bf16x2(z[6], z[7]);
        return pad_row ? make_uint4(0u, 0u, 0u, 0u) : v;
    }
    const float4 a0 = normal_quad_fast((uint32_t)(2 * ch), (uint32_t)row, matrix_id, sp.epoch, sp.round_key);
    const float4 a1 = normal_quad_fast((uint32_t)(2 * ch + 1), (uint32_t)row, matrix_id, sp.epoch, sp.round_key);
    v.x = pack_bf16x2(a0.x, a0.y); v.y = pack_bf16x2(a0.z, a0.w);
    v.z = pack_bf16x2(a1.x, a1.y); v.w = pack_bf16x2(a1.z, a1.w);
    return pad_row ? make_uint4(0u, 0u, 0u, 0u) : v;
}

__device__ __forceinline__ float sum_sq_bf16x8(const uint4& v)
{
    float a = 0.f;
    const uint32_t w[4] = { v.x, v.y, v.z, v.w };
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
        a = fmaf(lo, lo, a);
        a = fmaf(hi, hi, a);
    }
    return a;
}

__device__ __forceinline__ float fast_sqrt(float x)
{
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, const uint4& v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// 14 warps are allocated as 16: 128 registers per thread is the ceiling
__global__ void __launch_bounds__(TC_THREADS, 1)
project_tensor_kernel(const MatDesc* __restrict__ descs, const int* __restrict__ prefix, int n_mat, int tile_begin,
                      int tile_end, StepParams sp, TcTiling tl, int32_t* __restrict__ status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));

    const int r_slice = tl.r_slice, nblk = tl.nblk, stages = tl.stages;
    const bool staged = tl.staged != 0;
    const uint32_t stage_bytes = (uint32_t)(nblk * TC_BLOCK_BYTES + r_slice * 128);
    const uint32_t p_off = (uint32_t)(nblk * TC_BLOCK_BYTES);
    const uint32_t bars = smem_base + stages * stage_bytes;          // 8-byte mbarriers
    const uint32_t bar_g_full = bars, bar_p_full = bars + 32, bar_empty = bars + 64, bar_acc = bars + 96;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + stages * stage_bytes + 104);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + stages * stage_bytes + 108);
    const uint32_t bar_drain = bars + 112;
    volatile uint32_t* issued = reinterpret_cast<volatile uint32_t*>(smem_gen + stages * stage_bytes + 120);   // k-blocks the producer has requested
    float2* red = reinterpret_cast<float2*>(smem_gen + stages * stage_bytes + 256);          // [3][nblk*128]
    float* g2s = reinterpret_cast<float*>(smem_gen + stages * stage_bytes + 256 + 3 * 512 * 8);   // [8][nblk*128]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chan_tile = nblk * 128;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(bar_g_full + 8 * s, 1);
            ptx::mbar_init(bar_p_full + 8 * s, TC_GEN_THREADS / 32);
            ptx::mbar_init(bar_empty + 8 * s, 1 + TC_NORM_THREADS / 32);
        }
        ptx::mbar_init(bar_acc, 1);
        ptx::mbar_init(bar_drain, 1);
        *abort_flag = 0;
        *issued = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // k-block counter across tiles; its stage (it % stages) and phase ((it / stages) & 1) are kept
    // incrementally: a division per k-block is a large part of a single-thread role's instructions
    uint32_t it = 0, stage = 0, phase = 0;
    auto next_stage = [&]() { ++it; if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1; } };
    uint32_t tile_iter = 0;   // tiles done by this CTA: phase of the accumulator barrier

    for (int tile = tile_begin + blockIdx.x; tile < tile_end; tile += gridDim.x, ++tile_iter) {
        const int mat = find_matrix(prefix, n_mat, tile);
        // copy what the roles need into registers: the descriptor lives in global memory and
        // every shared-memory asm below is a compiler memory barrier
        const MatDesc* dp = descs + mat;
        const int tiles_k = __ldg(&dp->tiles_k);
        const int m = __ldg(&dp->m), n = __ldg(&dp->n);
        const bool tall = __ldg(&dp->tall) != 0;
        const uint32_t matrix_id = (uint32_t)__ldg(&dp->matrix_id);
        const void* tmap = dp->tmap;
        const void* tmap_p = dp->tmap_p;
        const float r_scale = __ldg(&dp->r_scale);
        float* const Mbase = dp->M;
        float* const Vbase = dp->V;
        float* const part = dp->part;
        float* const g2out = dp->g2;
        const int local = tile - __ldg(prefix + mat);
        const int tr = local % tiles_k, tn = local / tiles_k;   // row slices of one channel tile are neighbours
        const int j0 = tn * chan_tile, r0 = tr * r_slice;
        const int num_kb = (m + TC_BK - 1) / TC_BK;

        if (warp == 0) {
            // ---------------- TMA producer ----------------
            if (lane == 0) {
                ptx::fence_tensormap_acquire(tmap);
                if (staged) ptx::fence_tensormap_acquire(tmap_p);
                // G is read once in this pass, every CTA of a matrix reads the same P: tell L2 which to keep
                const uint64_t pol_g = ptx::policy_evict_first(), pol_p = ptx::policy_evict_last();
                for (int kb = 0; kb < num_kb; ++kb, next_stage()) {
                    const uint32_t s = stage, ph = phase;
                    if (!wait_phase(bar_empty + 8 * s, ph ^ 1, abort_flag, status)) break;
                    const uint32_t g_s = smem_base + s * stage_bytes;
                    ptx::mbar_arrive_expect_tx(bar_g_full + 8 * s,
                                               (uint32_t)(nblk * TC_BLOCK_BYTES + (staged ? r_slice * 128 : 0)));
                    if (staged) ptx::tma_load_2d_hint(g_s + p_off, tmap_p, kb * TC_BK, r0, bar_g_full + 8 * s, pol_p);
                    if (tall) {
                        for (int b = 0; b < nblk; ++b)
                            ptx::tma_load_2d_hint(g_s + b * TC_BLOCK_BYTES, tmap, kb * TC_BK, j0 + b * 128, bar_g_full + 8 * s, pol_g);
                    } else {
                        for (int b = 0; b < 2 * nblk; ++b)
                            ptx::tma_load_2d_hint(g_s + b * (TC_BLOCK_BYTES / 2), tmap, j0 + b * 64, kb * TC_BK, bar_g_full + 8 * s, pol_g);
                    }
                    *issued = it + 1;
                }
            }
            it = __shfl_sync(0xFFFFFFFFu, it, 0);     // after a wait gave up: the k-blocks requested so far
        } else if (warp == 1) {
            // ---------------- MMA issuer ----------------
            if (lane == 0) {
                const uint32_t idesc = ptx::instr_desc_bf16((uint32_t)r_slice, !tall);
                int kb = 0;
                for (; kb < num_kb; ++kb, next_stage()) {
                    const uint32_t s = stage, ph = phase;
                    if (!wait_phase(bar_g_full + 8 * s, ph, abort_flag, status)) break;
                    if (!staged && !wait_phase(bar_p_full + 8 * s, ph, abort_flag, status)) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t g_s = smem_base + s * stage_bytes, p_s = g_s + p_off;
                    for (int b = 0; b < nblk; ++b) {
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 16; ++kk) {
                            const uint64_t a_desc = tall
                                ? ptx::smem_desc_sw128(g_s + b * TC_BLOCK_BYTES + kk * 32, 16, 1024)
                                : ptx::smem_desc_sw128(g_s + b * TC_BLOCK_BYTES + kk * 2048, TC_BLOCK_BYTES / 2, 1024);
                            const uint64_t b_desc = ptx::smem_desc_sw128(p_s + kk * 32, 16, 1024);
                            ptx::mma_bf16(tmem_base + (uint32_t)(b * r_slice), a_desc, b_desc, idesc,
                                          (kb | kk) != 0 ? 1u : 0u);
                        }
                    }
                    ptx::mma_commit(bar_empty + 8 * s);
                }
                if (kb == num_kb) ptx::mma_commit(bar_acc);
            }
            it = __shfl_sync(0xFFFFFFFFu, it, 0);
        } else if (warp < 10) {
            // ---------------- generators: P tile for every k-block ----------------
            const int g = tid - 64;
            if (staged) {
                // P arrives by TMA from the scratch.  These warps instead ask L2 for the lines of G
                // TC_PREFETCH k-blocks ahead of the producer (into the next tile at the end of this one), so
                // that the loads into the shared-memory ring find them there.
                struct Ahead { const char* base; size_t pitch; int m, n, j0, nkb; bool tall; };
                auto ask = [&](const Ahead& a, int kb) {
                    for (int id = g; id < chan_tile; id += TC_GEN_THREADS) {
                        if (a.tall) {
                            if (a.j0 + id < a.n)
                                ptx::prefetch_l2(a.base + (size_t)(a.j0 + id) * a.pitch + (size_t)kb * (TC_BK * 2));
                        } else {
                            const int lines = chan_tile / 64;
                            const int row = kb * TC_BK + id / lines, col = a.j0 + (id % lines) * 64;
                            if (row < a.m && col < a.n)
                                ptx::prefetch_l2(a.base + (size_t)row * a.pitch + (size_t)col * 2);
                        }
                    }
                };
                const Ahead cur = { static_cast<const char*>(dp->gpad ? dp->gpad : dp->G),
                                    (size_t)__ldg(&dp->g_pitch) * 2, m, n, j0, num_kb, tall };
                Ahead nxt = cur;
                nxt.nkb = 0;
                const int next_tile = tile + (int)gridDim.x;
                if (tile_iter == 0)
                    for (int kb = 0; kb < TC_PREFETCH && kb < num_kb; ++kb) ask(cur, kb);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int want = kb + TC_PREFETCH;
                    if (want < num_kb) {
                        ask(cur, want);
                    } else if (next_tile < tile_end) {
                        if (want == num_kb || (kb == 0 && want > num_kb)) {
                            const int nm = find_matrix(prefix, n_mat, next_tile);
                            const MatDesc* q = descs + nm;
                            nxt.base = static_cast<const char*>(q->gpad ? q->gpad : q->G);
                            nxt.pitch = (size_t)__ldg(&q->g_pitch) * 2;
                            nxt.m = __ldg(&q->m); nxt.n = __ldg(&q->n); nxt.tall = __ldg(&q->tall) != 0;
                            nxt.j0 = ((next_tile - __ldg(prefix + nm)) / __ldg(&q->tiles_k)) * chan_tile;
                            nxt.nkb = (nxt.m + TC_BK - 1) / TC_BK;
                        }
                        if (want - num_kb < nxt.nkb) ask(nxt, want - num_kb);
                    }
                    // pacing only: nothing waits for these warps, so an expired wait costs nothing
                    for (uint32_t i = 0; i < TC_PACE_CAP && (int32_t)(*issued - it) <= 0 && !*abort_flag; ++i)
                        __nanosleep(100);
                }
            }
            for (int kb = 0; kb < num_kb && !staged; ++kb, next_stage()) {
                const uint32_t s = stage, ph = phase;
                if (!__all_sync(0xFFFFFFFFu, wait_phase(bar_empty + 8 * s, ph ^ 1, abort_flag, status))) break;
                const uint32_t p_s = smem_base + s * stage_bytes + p_off;
                // two rows per pass (32 rows apart) so that four Philox chains are in flight per thread
                const int total = r_slice * 8;
                for (int c = g; c < total; c += 2 * TC_GEN_THREADS) {
                    const int row = c >> 3, chunk = c & 7;
                    const uint32_t q0 = (uint32_t)(kb * (TC_BK / 4) + chunk * 2);
                    const uint32_t ka = (uint32_t)(r0 + row), kbrow = ka + 32u;
                    const uint32_t mid = matrix_id;
                    const float4 a0 = normal_quad_fast(q0, ka, mid, sp.epoch, sp.round_key);
                    const float4 a1 = normal_quad_fast(q0 + 1, ka, mid, sp.epoch, sp.round_key);
                    const float4 b0 = normal_quad_fast(q0, kbrow, mid, sp.epoch, sp.round_key);
                    const float4 b1 = normal_quad_fast(q0 + 1, kbrow, mid, sp.epoch, sp.round_key);
                    uint4 va, vb;
                    va.x = pack_bf16x2(a0.x, a0.y); va.y = pack_bf16x2(a0.z, a0.w);
                    va.z = pack_bf16x2(a1.x, a1.y); va.w = pack_bf16x2(a1.z, a1.w);
                    vb.x = pack_bf16x2(b0.x, b0.y); vb.y = pack_bf16x2(b0.z, b0.w);
                    vb.z = pack_bf16x2(b1.x, b1.y); vb.w = pack_bf16x2(b1.z, b1.w);
                    // padding rows of a rank that is not a multiple of 16
                    if (ka >= (uint32_t)sp.rank) va = make_uint4(0u, 0u, 0u, 0u);
                    if (kbrow >= (uint32_t)sp.rank) vb = make_uint4(0u, 0u, 0u, 0u);
                    const uint32_t at = p_s + row * 128 + ((chunk ^ (row & 7)) << 4);
                    st_shared_v4(at, va);
                    if (c + TC_GEN_THREADS < total) st_shared_v4(at + 32 * 128, vb);   // row + 32: same swizzle phase
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_p_full + 8 * s);
            }
        } else {
            // ---------------- column norms of G from the landed tiles ----------------
            const int t = tid - 320;
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            const int ccols = 16 * nblk;                 // wide: 16-byte chunk columns per stage
            const int parts = TC_NORM_THREADS / ccols;   // wide: threads sharing one chunk column
            const int cc = t % ccols, part = t / ccols;
            const int rows_pp = TC_BK / parts;
            for (int kb = 0; kb < num_kb; ++kb, next_stage()) {
                const uint32_t s = stage, ph = phase;
                if (!__all_sync(0xFFFFFFFFu, wait_phase(bar_g_full + 8 * s, ph, abort_flag, status))) break;   // the warp stays together
                const uint32_t g_s = smem_base + s * stage_bytes;
                if (tall) {
                    // block b, row t: 128 bytes = 8 chunks; the order of the chunks does not matter
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        if (b < nblk) {
                            const uint32_t row = g_s + b * TC_BLOCK_BYTES + t * 128;
#pragma unroll
                            for (int i = 0; i < 8; ++i) acc[b] += sum_sq_bf16x8(ld_shared_v4(row + (((i + t) & 7) << 4)));
                        }
                    }
                } else {
                    const uint32_t colbase = g_s + (cc >> 3) * (TC_BLOCK_BYTES / 2);
                    const int c = cc & 7;
                    for (int k = part * rows_pp; k < (part + 1) * rows_pp; ++k) {
                        const uint4 v = ld_shared_v4(colbase + k * 128 + ((c ^ (k & 7)) << 4));
                        const uint32_t w[4] = { v.x, v.y, v.z, v.w };
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
                            acc[2 * i] = fmaf(lo, lo, acc[2 * i]);
                            acc[2 * i + 1] = fmaf(hi, hi, acc[2 * i + 1]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_empty + 8 * s);
            }
            if (tall) {
#pragma unroll
                for (int b = 0; b < 4; ++b) if (b < nblk) g2s[b * 128 + t] = acc[b];
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) g2s[part * chan_tile + cc * 8 + e] = acc[e];
            }
        }

        if (warp >= 2) {
            // ---------------- epilogue: moments and per-channel sums ----------------
            const int q = warp & 3, widx = (warp - 2) >> 2;
            const int ch_in_blk = q * 32 + lane;
            for (int b = 0; b < nblk; ++b) red[widx * chan_tile + b * 128 + ch_in_blk] = make_float2(0.f, 0.f);
            const bool acc_ok = __all_sync(0xFFFFFFFFu, wait_phase(bar_acc, tile_iter & 1, abort_flag, status));   // tcgen05.ld needs the whole warp
            ptx::tc_fence_after_sync();
            const int chunks = r_slice / 16, items = acc_ok ? nblk * chunks : 0;
            float num = 0.f, den = 0.f;
            int cur_b = -1;
            for (int item = widx; item < items; item += 3) {
                const int b = item / chunks, cchunk = item % chunks;
                if (b != cur_b) {
                    if (cur_b >= 0) red[widx * chan_tile + cur_b * 128 + ch_in_blk] = make_float2(num, den);
                    cur_b = b; num = 0.f; den = 0.f;
                }
                float rv[16];
                ptx::tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * r_slice + cchunk * 16), rv);
                const int j = j0 + b * 128 + ch_in_blk;
                if (j < n && APOLLO_DBG_RANGE(state_at(true, 0, sp.rank_pad, r0 + cchunk * 16, j),
                                              state_at(true, 0, sp.rank_pad, r0 + cchunk * 16 + 15, j),
                                              state_elements(n, sp.rank_pad, true), status)) {
                    const int64_t at = state_at(true, 0, sp.rank_pad, r0 + cchunk * 16, j);     // channel blocks of 128: rows are 128 elements apart
                    const bool sb = sp.state_bf16 != 0;
                    float mv[16], vv[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        mv[k] = state_load(Mbase, at + (int64_t)k * 128, sb);
                        vv[k] = state_load(Vbase, at + (int64_t)k * 128, sb);
                    }
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const float r = rv[k] * r_scale;
                        const float mn = sp.beta1 * mv[k] + (1.0f - sp.beta1) * r;
                        const float vn = sp.beta2 * vv[k] + (1.0f - sp.beta2) * r * r;
                        state_store(Mbase, at + (int64_t)k * 128, mn, sb); state_store(Vbase, at + (int64_t)k * 128, vn, sb);
                        const float rt = __fdividef(mn * sp.inv_bc1, fast_sqrt(vn * sp.inv_bc2) + sp.eps);
                        num = fmaf(rt, rt, num);
                        den = fmaf(r, r, den);
                    }
                }
            }
            if (cur_b >= 0) red[widx * chan_tile + cur_b * 128 + ch_in_blk] = make_float2(num, den);
            ptx::tc_fence_before_sync();
            ptx::named_barrier(1, TC_EPI_THREADS);
            const int parts = tall ? 1 : TC_NORM_THREADS / (16 * nblk);
            for (int ch = tid - 64; ch < chan_tile; ch += TC_EPI_THREADS) {
                const int j = j0 + ch;
                if (j < n && APOLLO_DBG_RANGE((int64_t)tr * n + j, (int64_t)tr * n + j, (int64_t)__ldg(&dp->slices) * n, status)) {
                    const float2 a = red[ch], b2 = red[chan_tile + ch], c2 = red[2 * chan_tile + ch];
                    reinterpret_cast<float2*>(part)[(int64_t)tr * n + j] = make_float2(a.x + b2.x + c2.x, a.y + b2.y + c2.y);
                    if (tr == 0) {
                        float g2 = 0.f;
                        for (int p = 0; p < parts; ++p) g2 += g2s[p * chan_tile + ch];
                        g2out[j] = g2;
                    }
                }
            }
        }
        // the accumulator is drained: the issuer may start the next tile.  After a wait gave up, all
        // warps of the barrier leave together; the producer leaves on its own
        if (warp >= 1) {
            ptx::tc_fence_before_sync();
            const bool stop = ptx::named_barrier_or(2, TC_THREADS - 32, *abort_flag != 0);
            ptx::tc_fence_after_sync();
            if (stop) break;
        } else if (__shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0) {
            break;
        }
    }

    // Whatever is still in flight lands before shared memory and TMEM are given up.  On the normal
    // path every load was consumed and every MMA committed, so these waits return at once.
    if (tid == 0) {
        for (uint32_t s = 0; s < (uint32_t)stages && s < it; ++s) {
            const uint32_t last = s + (it - 1 - s) / stages * stages;    // last k-block requested into stage s
            drain_phase(bar_g_full + 8 * s, (last / stages) & 1);
        }
    }
    if (tid == 32) {
        ptx::mma_commit(bar_drain);
        drain_phase(bar_drain, 0);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, 512);
}

// ----------------------------------------------------------------------------------------
// Pair kernel (default): two CTAs of a cluster share every MMA (cta_group::2,
// M = 256).  A pair tile is 256 channels x r_slice rows of R.  Each CTA loads the G tile of its own
// 128 channels and half of the rows of the P tile (so a k-block costs 32 KB of shared-memory fill per
// CTA instead of 48 KB for the same work), and keeps r_slice accumulator columns per buffer, double
// buffered: the epilogue of one tile runs under the main loop of the next.
//   warp 0      G producer, warp 2  P producer: the TMA loads of both CTAs count their bytes on the
//               LEADER's `full` barrier of the stage
//   warp 1      leader only: MMA issuer; its commits are multicast to both CTAs
//   warps 4-7   squared column norms of this CTA's G tile, after the MMA that read it has finished
//   warps 8-15  epilogue of this CTA's 128 channels
// Barriers per stage s: full[s] (leader: one arrive.expect_tx for the bytes of both CTAs),
// done[s] (both: the leader's commit), empty[s] (both: the four norm warps).
// Shared memory holds nothing but the ring and the barriers (seven 32 KB stages at r_slice = 256):
// the per-channel partial sums go to global memory as slices that finalize_kernel adds up, one
// per half of the epilogue warps and, for wide matrices, one per norm warp.
// ----------------------------------------------------------------------------------------
constexpr int P2_THREADS = 512;
constexpr int P2_G_BYTES = 128 * TC_BK * 2;        // G of 128 channels, one k-block: 16 KiB
constexpr int P2_MAX_STAGES = 8;
constexpr int P2_MISC_BYTES = 512 + 1024;          // barriers and flags, alignment slack
static_assert(P2_MISC_BYTES == 1536, "tensor_path_configure() reserves this many bytes");

// RAW: the list has matrices whose G tiles are re-aligned in shared memory (TcTiling::raw).  The kernel without
// that code is a separate instantiation, so that lists without such matrices run exactly the code they ran
// before it existed (with it compiled in, the other roles of the kernel came out 15 % slower).
// SPLIT: the gradients are fp32 (TcTiling::split).  A tile's contraction then runs over three segments of the
// bfloat16 high/low copies, P_hi G_hi + P_lo G_hi + P_hi G_lo (what is dropped, P_lo G_lo, is 2^-16 of a
// term), and the column norms come from the kernel that made the copies.  A third instantiation, for the
// same reason as the second.
// SB16: M and V are stored as bfloat16 (StepParams::state_bf16) -- a compile-time fact of the epilogue: as a run-time
// flag on every load and store it cost the fp32 lists up to 4 % of the pass.
template <bool RAW, bool SPLIT, bool SB16>
__global__ void __launch_bounds__(P2_THREADS, 1)
project_pair_kernel(const MatDesc* __restrict__ descs, const int* __restrict__ prefix, int n_mat, int tile_begin,
                    int tile_end, StepParams sp, TcTiling tl, GenArgs gen, int32_t* __restrict__ status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));

    const uint32_t rank = ptx::cluster_ctarank();          // 0: leader, 1: peer
    const int r_slice = tl.r_slice, ns = tl.stages, r_half = r_slice / 2;
    // the G part of a stage holds 128 channels x 64 rows in the UMMA layout (16 KiB); in a list with matrices
    // whose rows start on no 16-byte boundary it is large enough for the 64 row pieces as fetched (17 KiB)
    const uint32_t g_bytes = RAW ? (uint32_t)RAW_G_BYTES : (uint32_t)P2_G_BYTES;
    const uint32_t p_bytes = (uint32_t)r_half * 128u, stage_bytes = g_bytes + p_bytes;
    const uint32_t misc = (uint32_t)ns * stage_bytes;
    const uint32_t bars = smem_base + misc;
    const uint32_t bar_full = bars, bar_done = bars + 64, bar_empty = bars + 128, bar_acc_full = bars + 192,
                   bar_acc_empty = bars + 208, bar_drain = bars + 224, bar_raw = bars + 256, bar_read = bars + 320,
                   bar_ready = bars + 384;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + misc + 240);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + misc + 244);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < ns; ++s) {
            ptx::mbar_init(bar_full + 8 * s, 1);        // the leader's arrive.expect_tx
            ptx::mbar_init(bar_done + 8 * s, 1);        // the leader's commit
            ptx::mbar_init(bar_empty + 8 * s, 4);       // four norm warps of this CTA
            // used by re-aligned tiles only; these complete one phase per such k-block, not per turn of the ring,
            // so whoever waits on them keeps the parity of each stage's next phase in a bit mask of its own
            ptx::mbar_init(bar_raw + 8 * s, 1);         // this CTA's arrive.expect_tx for the row pieces as fetched
            ptx::mbar_init(bar_read + 8 * s, 4);        // the four norm warps have the row pieces in registers
            ptx::mbar_init(bar_ready + 8 * s, 8);       // leader's copy: the norm warps of both CTAs have written the tile
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(bar_acc_full + 8 * b, 1);    // the leader's commit
            ptx::mbar_init(bar_acc_empty + 8 * b, 16);  // eight epilogue warps of each CTA (the leader's copy is used)
        }
        ptx::mbar_init(bar_drain, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_addr(tmem_slot), 512);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();          // both CTAs' barriers exist before any remote arrive, remote byte count or multicast commit
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // k-block and tile counters of this role; the stage index and phase of k-block `it` are kept
    // incrementally (stage = it % ns, phase = (it / ns) & 1): the single-thread roles are bound by
    // their own instruction count, and a division per k-block is a large part of it
    uint32_t it = 0, tile_iter = 0, stage = 0, phase = 0;
    auto next_stage = [&]() { ++it; if (++stage == (uint32_t)ns) { stage = 0; phase ^= 1; } };
    uint32_t raw_bits = 0, raw_used = 0;     // bit s: parity of stage s's next re-aligned k-block; stages that had one

    // ---------------- generator warps (TcTiling::gen): P of every matrix of the launch, ahead of its use ----------------
    // The spare warps of all CTAs (warp 3 everywhere, warp 1 of the peers, whose MMA role is the leader's) draw
    // tickets; a ticket is one of GEN_CHUNKS pieces of one matrix's P, written as 16-byte vectors into the
    // matrix's slot of the scratch (a ring of `slots` slots over the matrices in list order).  A slot is
    // rewritten once every tile of its previous user has finished its MMAs (use_done); the P producers of
    // the tiles wait for all pieces of their matrix (gen_done).  The lowest ticket outstanding never waits
    // on anything that is not already under way, so the scheme cannot deadlock; every wait is bounded.
    if (tl.gen != 0 && (warp == 3 || (warp == 1 && rank == 1))) {
        for (;;) {
            uint32_t ticket = 0;
            if (lane == 0) ticket = atomicAdd(gen.ticket, 1u);
            ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
            const int q = gen.q_begin + (int)(ticket / GEN_CHUNKS);
            if (q >= gen.q_end) break;
            const int piece = (int)(ticket % GEN_CHUNKS);
            const int gm = __ldg(gen.mats + q);
            int ok = 1;
            if (q - tl.slots >= gen.q_begin) {
                const int pm = __ldg(gen.mats + q - tl.slots);
                const uint32_t need = (uint32_t)(__ldg(&descs[pm].tiles_n) * __ldg(&descs[pm].tiles_k));
                if (lane == 0) ok = wait_counter(gen.use_done + pm, need, abort_flag, status, 112) ? 1 : 0;
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
            }
            if (!ok) break;
            const MatDesc* gp = descs + gm;
            const int half_vpr = __ldg(&gp->m_pad) / 8;
            const int vec_per_row = SPLIT ? 2 * half_vpr : half_vpr, total = sp.rank_pad * vec_per_row;
            const int per = (total + GEN_CHUNKS - 1) / GEN_CHUNKS;
            const int c_end = min(total, (piece + 1) * per);
            const uint32_t matrix_id = (uint32_t)__ldg(&gp->matrix_id);
            const float* __restrict__ ext_p = gp->ext_p;
            const int gmm = __ldg(&gp->m);
            uint4* const out = static_cast<uint4*>(gp->pstage);
            // two vectors per pass: four Philox chains in flight per thread
            for (int c = piece * per + lane; c < c_end; c += 64) {
                if (!APOLLO_DBG_RANGE(c, c, total, status)) break;
                const int row0 = c / vec_per_row;
                const uint4 v0 = p_vector<SPLIT>(ext_p, gmm, row0, c - row0 * vec_per_row, matrix_id, sp, half_vpr);
                if (c + 32 < c_end) {
                    const int row1 = (c + 32) / vec_per_row;
                    out[c + 32] = p_vector<SPLIT>(ext_p, gmm, row1, c + 32 - row1 * vec_per_row, matrix_id, sp, half_vpr);
                }
                out[c] = v0;
            }
            ptx::fence_proxy_async_global();
            __threadfence();
            __syncwarp();
            if (lane == 0) red_release_gpu_add(gen.gen_done + gm, 1u);
        }
    }

    const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;
    int mat = find_matrix(prefix, n_mat, tile_begin + pair < tile_end ? tile_begin + pair : tile_begin);
    int p_ready_mat = -1;      // P producer: the matrix whose generated P it has already waited for
    for (int tile = tile_begin + pair; tile < tile_end; tile += pairs, ++tile_iter) {
        // the tiles of a CTA come in increasing order: the matrix index only moves forward
        while (mat + 1 < n_mat && __ldg(prefix + mat + 1) <= tile) ++mat;
        const MatDesc* dp = descs + mat;
        const int tiles_k = __ldg(&dp->tiles_k);
        const int m = __ldg(&dp->m), n = __ldg(&dp->n);
        const bool tall = __ldg(&dp->tall) != 0;
        const int local = tile - __ldg(prefix + mat);
        const int tr = local % tiles_k, tn = local / tiles_k;
        const int j0 = tn * 256 + (int)rank * 128, r0 = tr * r_slice;
        const int nkb1 = (m + TC_BK - 1) / TC_BK;
        const int num_kb = SPLIT ? 3 * nkb1 : nkb1;
        // SPLIT: where k-block kb starts along the projected side of the G copy ([hi; lo], m_pad apart) and of the
        // P slot ([P_hi | P_lo]): segments hi x hi, lo x hi, hi x lo (P x G)
        const int m_pad_s = SPLIT ? __ldg(&dp->m_pad) : 0;
        auto g_at = [&](int kb) { return SPLIT ? (kb >= 2 * nkb1 ? m_pad_s + (kb - 2 * nkb1) * TC_BK : (kb >= nkb1 ? kb - nkb1 : kb) * TC_BK) : kb * TC_BK; };
        auto p_at = [&](int kb) { return SPLIT ? (kb >= 2 * nkb1 ? (kb - 2 * nkb1) * TC_BK : (kb >= nkb1 ? m_pad_s + (kb - nkb1) * TC_BK : kb * TC_BK)) : kb * TC_BK; };
        const uint32_t buf = tile_iter & 1, use = tile_iter >> 1;
        // this matrix's rows start on no 16-byte boundary: its tiles are fetched as they lie and re-aligned by the norm warps
        const bool raw_tile = RAW && __ldg(&dp->raw) != 0;

        if (warp == 0) {
            // ---------------- G producer (one thread in each CTA) ----------------
            if (lane == 0) {
                const void* tmap = dp->tmap;
                ptx::fence_tensormap_acquire(tmap);
                // G is read once per row slice: with one slice it may leave L2 at once; with several, the pairs
                // that work on the other slices of this channel tile at about the same time should find it there
                const uint64_t pol_g = tiles_k > 1 ? ptx::policy_evict_normal() : ptx::policy_evict_first();
                // the bytes of both CTAs are counted on the leader's barrier; the peer's may arrive
                // there before the leader's expect_tx (the count is signed), never a phase early,
                // because the peer's stage is only free once the leader's MMA has consumed it
                const uint32_t full0 = ptx::map_to_cta(bar_full, 0);
                const int cols = __ldg(&dp->cols);
                for (int kb = 0; kb < num_kb; ++kb, next_stage()) {
                    const uint32_t s = stage;
                    // with re-aligned tiles in the list the norm warps free a stage before the MMA has read it
                    if (RAW && !wait_phase(bar_done + 8 * s, phase ^ 1, abort_flag, status, 101)) break;
                    if (!wait_phase(bar_empty + 8 * s, phase ^ 1, abort_flag, status, 102)) break;
                    const uint32_t g_s = smem_base + s * stage_bytes, full = full0 + 8 * s;
                    if (raw_tile) {
                        // 8 boxes, one per row residue b: RAW_BOX_W elements of rows 8 a + b, a = 8 kb .. 8 kb + 7,
                        // starting at the 16-byte unit that holds channel j0 of those rows; they land on this CTA's
                        // own barrier, the leader's `full` barrier expects the P bytes only
                        ptx::mbar_arrive_expect_tx(bar_raw + 8 * s, (uint32_t)RAW_G_BYTES);
                        raw_bits ^= 1u << s; raw_used |= 1u << s;
                        if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * s, 2u * p_bytes);
#pragma unroll
                        for (int b = 0; b < 8; ++b)
                            ptx::tma_load_2d_hint(g_s + b * (8 * RAW_BOX_W * 2), tmap, (b * cols + j0) & ~7, kb * 8,
                                                  bar_raw + 8 * s, pol_g);
                        continue;
                    }
                    if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * s, 2u * (P2_G_BYTES + p_bytes));   // G and P of both CTAs
                    if (tall) {
                        ptx::tma_load_2d_pair(g_s, tmap, g_at(kb), j0, full, pol_g);
                    } else {
                        ptx::tma_load_2d_pair(g_s, tmap, j0, g_at(kb), full, pol_g);
                        ptx::tma_load_2d_pair(g_s + P2_G_BYTES / 2, tmap, j0 + 64, g_at(kb), full, pol_g);
                    }
                }
            }
            __syncwarp();
            if (__shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0) break;
        } else if (warp == 2) {
            // ---------------- P producer (one thread in each CTA): this CTA's half of the rows, same stage, same barrier ----------------
            if (lane == 0) {
                const void* tmap_p = dp->tmap_p;
                ptx::fence_tensormap_acquire(tmap_p);
                const uint64_t pol_p = ptx::policy_evict_last();
                const uint32_t full0 = ptx::map_to_cta(bar_full, 0);
                const int p_row = r0 + (int)rank * r_half;
                bool p_ok = true;
                if (tl.gen != 0 && mat != p_ready_mat) {
                    // every piece of this matrix's P has been written (by generic stores of other SMs): order
                    // them before this thread's loads through the async proxy
                    p_ok = wait_counter(gen.gen_done + mat, (uint32_t)GEN_CHUNKS, abort_flag, status, 105);
                    ptx::fence_proxy_async_global();
                    p_ready_mat = mat;
                }
                for (int kb = 0; p_ok && kb < num_kb; ++kb, next_stage()) {
                    const uint32_t s = stage;
                    // The P part of a stage is read by the MMA alone.  Without re-aligned tiles in the list `empty`
                    // (the norm warps, who wait for the MMA) says that it is free; with them the norm warps may
                    // free a stage before this thread has even filled it, and the MMA's own commit is the signal.
                    if (RAW ? !wait_phase(bar_done + 8 * s, phase ^ 1, abort_flag, status, 103)
                            : !wait_phase(bar_empty + 8 * s, phase ^ 1, abort_flag, status, 104)) break;
                    ptx::tma_load_2d_pair(smem_base + s * stage_bytes + g_bytes, tmap_p, p_at(kb), p_row, full0 + 8 * s, pol_p);
                }
            }
            __syncwarp();
            if (__shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0) break;
        } else if (warp == 1) {
            // ---------------- MMA issuer (leader only) ----------------
            if (lane == 0 && rank == 0) {
                const uint32_t idesc = ptx::instr_desc_bf16((uint32_t)r_slice, !tall, 256u);
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)r_slice;
                bool ok = wait_phase(bar_acc_empty + 8 * buf, (use & 1) ^ 1, abort_flag, status, 106);   // epilogue of the tile before last
                ptx::tc_fence_after_sync();
                // descriptors of stage 0, k-step 0; the start-address field (bits 0..13, address >> 4) is the
                // only one that moves, and shared-memory addresses stay below 2^18, so it never carries out
                const uint64_t a_desc0 = tall ? ptx::smem_desc_sw128(smem_base, 16, 1024)
                                              : ptx::smem_desc_sw128(smem_base, P2_G_BYTES / 2, 1024);
                const uint64_t b_desc0 = ptx::smem_desc_sw128(smem_base + g_bytes, 16, 1024);
                const uint32_t a_step = tall ? 32u >> 4 : 2048u >> 4, stage_step = stage_bytes >> 4;
                int kb = 0;
                for (; ok && kb < num_kb; ++kb, next_stage()) {
                    const uint32_t s = stage;
                    if (!wait_phase(bar_full + 8 * s, phase, abort_flag, status, 107)) break;
                    if (raw_tile) {        // the G tile was written by the norm warps of both CTAs
                        if (!wait_phase(bar_ready + 8 * s, (raw_bits >> s) & 1u, abort_flag, status, 113)) break;
                        raw_bits ^= 1u << s;
                    }
                    ptx::tc_fence_after_sync();
                    const uint64_t a_desc = a_desc0 + s * stage_step, b_desc = b_desc0 + s * stage_step;
#pragma unroll
                    for (int kk = 0; kk < TC_BK / 16; ++kk)
                        ptx::mma_bf16_pair(d_tmem, a_desc + kk * a_step, b_desc + kk * 2, idesc, (kb | kk) != 0 ? 1u : 0u);
                    ptx::mma_commit_pair(bar_done + 8 * s, 3);
                }
                if (ok && kb == num_kb) ptx::mma_commit_pair(bar_acc_full + 8 * buf, 3);
            }
            __syncwarp();
            if (__shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0) break;
        } else if (warp >= 4 && warp < 8) {
            // ---------------- squared column norms of this CTA's 128 channels ----------------
            const int t = tid - 128;
            // packed pairs of fp32 accumulators (fma.rn.f32x2).  wide: acc2[i] = channels 2i, 2i+1 of this
            // thread's eight; tall: acc2[4 pass + i] = word i of the 16-byte chunks of row unit `pass`
            uint64_t acc2[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc2[e] = 0ull;
            const int cc = t & 15, part = t >> 4;     // wide: 16 chunk columns x 8 row groups
            const uint32_t ready_leader = ptx::map_to_cta(bar_ready, 0);
            const int cols = __ldg(&dp->cols);
            for (int kb = 0; kb < num_kb; ++kb, next_stage()) {
                const uint32_t s = stage, ph = phase;
                const uint32_t g_s = smem_base + s * stage_bytes;
                if (raw_tile) {
                    // ---- re-align the row pieces as fetched into the UMMA layout, in place, before the MMA ----
                    // The stage holds 8 boxes (row residue b) of 8 rows (a) of RAW_BOX_W elements; row 8 a + b of the
                    // k-block starts (b cols + j0) mod 8 elements into its piece.  This warp takes the residues
                    // 2 (warp - 4) and + 1; a lane takes one 16-byte chunk column c of one 64-channel half h for two
                    // rows a per (b, h): a quarter-warp reads 128 contiguous bytes of one piece and writes the eight
                    // chunks of one row of the swizzled tile (no bank conflicts either way).  All pieces are read into
                    // registers (and shifted into place there) before the first write: the tile overwrites them.
                    const uint32_t rph = (raw_bits >> s) & 1u;
                    raw_bits ^= 1u << s;
                    const bool ok = __all_sync(0xFFFFFFFFu, wait_phase(bar_raw + 8 * s, rph, abort_flag, status, 108));
                    const int c = lane & 7, a_lo = lane >> 3;
                    uint4 o[8];
                    if (ok) {
                        // one row residue (four passes) at a time: its eight 16-byte loads are issued together, and the
                        // shift is done without a branch (the word part of the offset by selects, the half-word part by
                        // the funnel shift), so that nothing keeps the loads of the second residue from overlapping it
#pragma unroll
                        for (int bsel = 0; bsel < 2; ++bsel) {
                            const int b = 2 * (warp - 4) + bsel;
                            uint4 lo[4], hi[4];
#pragma unroll
                            for (int p4 = 0; p4 < 4; ++p4) {
                                const int h = p4 >> 1, a = a_lo + 4 * (p4 & 1);
                                const uint32_t src = g_s + (uint32_t)((b * 8 + a) * (RAW_BOX_W * 2) + (h * 8 + c) * 16);
                                lo[p4] = ld_shared_v4(src);
                                hi[p4] = ld_shared_v4(src + 16);
                            }
                            const uint32_t mis = (uint32_t)((b * cols + j0) & 7) * 2u, wsel = mis >> 2, sh = (mis & 2u) * 8u;
                            const bool s1 = wsel >= 1u, s2 = wsel >= 2u, s3 = wsel >= 3u;
#pragma unroll
                            for (int p4 = 0; p4 < 4; ++p4) {
                                const uint32_t w[8] = { lo[p4].x, lo[p4].y, lo[p4].z, lo[p4].w, hi[p4].x, hi[p4].y, hi[p4].z, hi[p4].w };
                                uint32_t u[5];       // words wsel .. wsel + 4 of the piece
#pragma unroll
                                for (int k = 0; k < 5; ++k) u[k] = s2 ? (s3 ? w[k + 3] : w[k + 2]) : (s1 ? w[k + 1] : w[k]);
                                o[4 * bsel + p4] = make_uint4(__funnelshift_r(u[0], u[1], sh), __funnelshift_r(u[1], u[2], sh),
                                                              __funnelshift_r(u[2], u[3], sh), __funnelshift_r(u[3], u[4], sh));
                            }
                        }
                        // channels at and beyond the end of the row hold the next row's elements: zero them (last channel tile only)
                        if (j0 + 128 > cols) {
#pragma unroll
                            for (int pass = 0; pass < 8; ++pass) {
                                const int jc = j0 + ((pass >> 1) & 1) * 64 + c * 8;
                                uint32_t v[4] = { o[pass].x, o[pass].y, o[pass].z, o[pass].w };
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    if (jc + 2 * k >= cols) v[k] = 0u;
                                    else if (jc + 2 * k + 1 >= cols) v[k] &= 0xFFFFu;
                                }
                                o[pass] = make_uint4(v[0], v[1], v[2], v[3]);
                            }
                        }
                    }
                    // all four norm warps have read before anyone writes (a bounded wait like every other: a warp
                    // that gave up does not arrive, and the others give up in turn)
                    __syncwarp();
                    if (!ok) break;
                    if (lane == 0) ptx::mbar_arrive(bar_read + 8 * s);
                    // the column norms need only the registers: they fill the wait for the other three warps
                    if (tr == 0) {
#pragma unroll
                        for (int pass = 0; pass < 8; ++pass) {
                            const int h = (pass >> 1) & 1;
                            ptx::fma_sq_f32x2(acc2[h * 4 + 0], ptx::bf16x2_to_f32x2(o[pass].x));
                            ptx::fma_sq_f32x2(acc2[h * 4 + 1], ptx::bf16x2_to_f32x2(o[pass].y));
                            ptx::fma_sq_f32x2(acc2[h * 4 + 2], ptx::bf16x2_to_f32x2(o[pass].z));
                            ptx::fma_sq_f32x2(acc2[h * 4 + 3], ptx::bf16x2_to_f32x2(o[pass].w));
                        }
                    }
                    if (!__all_sync(0xFFFFFFFFu, wait_phase(bar_read + 8 * s, rph, abort_flag, status, 109))) break;
#pragma unroll
                    for (int pass = 0; pass < 8; ++pass) {
                        const int b = 2 * (warp - 4) + (pass >> 2), h = (pass >> 1) & 1, a = a_lo + 4 * (pass & 1);
                        const int krow = 8 * a + b;      // row of the k-block
                        st_shared_v4(g_s + (uint32_t)(h * (P2_G_BYTES / 2) + krow * 128 + ((c ^ (krow & 7)) << 4)), o[pass]);
                    }
                    ptx::fence_proxy_async_smem();      // the tile was written by plain stores; the MMA reads it through the async proxy
                    __syncwarp();
                    if (lane == 0) {
                        ptx::mbar_arrive_remote(ready_leader + 8 * s);
                        ptx::mbar_arrive(bar_empty + 8 * s);      // the producers also wait for the MMA's commit before refilling
                    }
                    continue;
                }
                if (!__all_sync(0xFFFFFFFFu, wait_phase(bar_done + 8 * s, ph, abort_flag, status, 110))) break;   // landed, and the MMA has read it
                if (tr != 0 || SPLIT) {
                    // the norms belong to the channel tile, not to the row slice: the first slice has them
                    // (and those of an fp32 gradient come from the kernel that split it)
                } else if (tall) {
                    // units (row, half): 256 units over 128 threads; the order of the chunks is free
#pragma unroll
                    for (int pass = 0; pass < 2; ++pass) {
                        const int u = t + pass * 128, row = u >> 1, half = u & 1;
                        const uint32_t base = g_s + row * 128 + half * 64;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint4 v = ld_shared_v4(base + (((i + row) & 3) << 4));
                            ptx::fma_sq_f32x2(acc2[4 * pass + 0], ptx::bf16x2_to_f32x2(v.x));
                            ptx::fma_sq_f32x2(acc2[4 * pass + 1], ptx::bf16x2_to_f32x2(v.y));
                            ptx::fma_sq_f32x2(acc2[4 * pass + 2], ptx::bf16x2_to_f32x2(v.z));
                            ptx::fma_sq_f32x2(acc2[4 * pass + 3], ptx::bf16x2_to_f32x2(v.w));
                        }
                    }
                } else {
                    const uint32_t colbase = g_s + (cc >> 3) * (P2_G_BYTES / 2);
                    const int c = cc & 7;
#pragma unroll
                    for (int i8 = 0; i8 < 8; ++i8) {
                        const int k = part + 8 * i8;
                        const uint4 v = ld_shared_v4(colbase + k * 128 + ((c ^ (k & 7)) << 4));
                        ptx::fma_sq_f32x2(acc2[0], ptx::bf16x2_to_f32x2(v.x));
                        ptx::fma_sq_f32x2(acc2[1], ptx::bf16x2_to_f32x2(v.y));
                        ptx::fma_sq_f32x2(acc2[2], ptx::bf16x2_to_f32x2(v.z));
                        ptx::fma_sq_f32x2(acc2[3], ptx::bf16x2_to_f32x2(v.w));
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_empty + 8 * s);
            }
            // squared norms of this tile's channels -> global slices (only the first row slice writes them)
            const bool stop = __shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0;     // one answer per warp
            float* const g2out = dp->g2;
            if (raw_tile) {
                // lanes with the same chunk column (lane & 7) hold the rows a = lane >> 3 (+ 4) of the same 16 channels:
                // 8 of half 0 in acc2[0..3], 8 of half 1 in acc2[4..7]; one slice per warp (its two row residues)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float x0, x1;
                    ptx::f32x2_unpack(acc2[i], x0, x1);
                    x0 += __shfl_xor_sync(0xFFFFFFFFu, x0, 8);  x1 += __shfl_xor_sync(0xFFFFFFFFu, x1, 8);
                    x0 += __shfl_xor_sync(0xFFFFFFFFu, x0, 16); x1 += __shfl_xor_sync(0xFFFFFFFFu, x1, 16);
                    const int j = j0 + (i >> 2) * 64 + (lane & 7) * 8 + 2 * (i & 3);
                    if (!stop && !SPLIT && tr == 0 && lane < 8) {
                        float* const out = g2out + (int64_t)(warp - 4) * n;
                        if (j < n && APOLLO_DBG_RANGE((int64_t)(warp - 4) * n + j, (int64_t)(warp - 4) * n + j, (int64_t)__ldg(&dp->g2_slices) * n, status)) out[j] = x0;
                        if (j + 1 < n && APOLLO_DBG_RANGE((int64_t)(warp - 4) * n + j + 1, (int64_t)(warp - 4) * n + j + 1, (int64_t)__ldg(&dp->g2_slices) * n, status)) out[j + 1] = x1;
                    }
                }
            } else if (tall) {
                // lanes 2k and 2k+1 hold the two halves of one stored row
#pragma unroll
                for (int pass = 0; pass < 2; ++pass) {
                    const float mine = (ptx::f32x2_sum(acc2[4 * pass]) + ptx::f32x2_sum(acc2[4 * pass + 1])) +
                                       (ptx::f32x2_sum(acc2[4 * pass + 2]) + ptx::f32x2_sum(acc2[4 * pass + 3]));
                    const float v = mine + __shfl_xor_sync(0xFFFFFFFFu, mine, 1);
                    const int j = j0 + ((t + pass * 128) >> 1);
                    if (!stop && !SPLIT && tr == 0 && !(lane & 1) && j < n &&
                        APOLLO_DBG_RANGE(j, j, (int64_t)__ldg(&dp->g2_slices) * n, status))
                        g2out[j] = v;
                }
            } else {
                // lanes l and l + 16 hold two row groups of the same eight channels: one slice per warp
                float acc[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) ptx::f32x2_unpack(acc2[i], acc[2 * i], acc[2 * i + 1]);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float v = acc[e] + __shfl_xor_sync(0xFFFFFFFFu, acc[e], 16);
                    const int j = j0 + cc * 8 + e;
                    if (!stop && !SPLIT && tr == 0 && lane < 16 && j < n &&
                        APOLLO_DBG_RANGE((int64_t)(warp - 4) * n + j, (int64_t)(warp - 4) * n + j, (int64_t)__ldg(&dp->g2_slices) * n, status))
                        g2out[(int64_t)(warp - 4) * n + j] = v;
                }
            }
            if (stop) break;
        } else if (warp >= 8) {
            // ---------------- epilogue of this tile, under the main loop of the next ----------------
            const int q = warp & 3, half = (warp - 8) >> 2;
            const int ch = q * 32 + lane, j = j0 + ch;
            float* const Mbase = dp->M;
            float* const Vbase = dp->V;
            const float r_scale = __ldg(&dp->r_scale);
            // One chunk ahead of its loads, the warp asks L2 for the 32 lines of the chunk (lane l: row l of M,
            // lane 16 + l: row l of V, the warp's 32 channels): the loads then pay an L2 round trip, and twice
            // as many bytes of the moments are in flight per SM.  The first chunk is asked for before the
            // wait for the accumulator.
            // M and V are stored in channel blocks of 128 (state_at): this CTA's block, rows 128 elements apart
            const int64_t tile_el = (int64_t)(j0 >> 7) * sp.rank_pad * 128;
            const bool pf = tl.epi_prefetch != 0 && j0 + q * 32 < n;
            const char* const pf_base = reinterpret_cast<const char*>(lane < 16 ? Mbase : Vbase);
            const int64_t pf_esz = SB16 ? 2 : 4;
            auto ask = [&](int chunk) {
                ptx::prefetch_l2(pf_base + (tile_el + (int64_t)(r0 + chunk * 16 + (lane & 15)) * 128 + q * 32) * pf_esz);
            };
            const int pf_d = tl.epi_prefetch;                            // distance in chunks of this warp
            if (pf)
                for (int a = 0; a < pf_d; ++a)
                    if (half + 2 * a < r_slice / 16) ask(half + 2 * a);
            const bool acc_ok = __all_sync(0xFFFFFFFFu, wait_phase_idle(bar_acc_full + 8 * buf, use & 1, abort_flag, status, 111));   // tcgen05.ld needs the whole warp
            ptx::tc_fence_after_sync();
            // the MMAs of this tile are done, so both CTAs' last P tiles have been read: one count per pair tile
            if (tl.gen != 0 && rank == 0 && warp == 8 && lane == 0 && acc_ok) red_release_gpu_add(gen.use_done + mat, 1u);
            float num = 0.f, den = 0.f;
            const int chunks = acc_ok ? r_slice / 16 : 0;
            for (int cchunk = half; cchunk < chunks; cchunk += 2) {
                if (pf && cchunk + 2 * pf_d < chunks) ask(cchunk + 2 * pf_d);
                float rv[16];
                ptx::tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)r_slice + (uint32_t)(cchunk * 16), rv);
                if (j < n && APOLLO_DBG_RANGE(tile_el + (int64_t)(r0 + cchunk * 16) * 128 + ch,
                                              tile_el + (int64_t)(r0 + cchunk * 16 + 15) * 128 + ch,
                                              state_elements(n, sp.rank_pad, true), status)) {
                    const int64_t at = tile_el + (int64_t)(r0 + cchunk * 16) * 128 + ch;
                    constexpr bool sb = SB16;
                    float mv[16], vv[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        mv[k] = state_load(Mbase, at + (int64_t)k * 128, sb);
                        vv[k] = state_load(Vbase, at + (int64_t)k * 128, sb);
                    }
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const float r = rv[k] * r_scale;
                        const float mn = sp.beta1 * mv[k] + (1.0f - sp.beta1) * r;
                        const float vn = sp.beta2 * vv[k] + (1.0f - sp.beta2) * r * r;
                        state_store(Mbase, at + (int64_t)k * 128, mn, sb); state_store(Vbase, at + (int64_t)k * 128, vn, sb);
                        const float rt = __fdividef(mn * sp.inv_bc1, fast_sqrt(vn * sp.inv_bc2) + sp.eps);
                        num = fmaf(rt, rt, num);
                        den = fmaf(r, r, den);
                    }
                }
            }
            // this warp has read its share of the accumulator: hand the buffer back to the issuer
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0 && acc_ok) ptx::mbar_arrive_remote(ptx::map_to_cta(bar_acc_empty + 8 * buf, 0));
            if (acc_ok && j < n &&
                APOLLO_DBG_RANGE((int64_t)(tr * 2 + half) * n + j, (int64_t)(tr * 2 + half) * n + j, (int64_t)__ldg(&dp->slices) * n, status))
                reinterpret_cast<float2*>(dp->part)[(int64_t)(tr * 2 + half) * n + j] = make_float2(num, den);
            if (__shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0) break;
        } else if (__shfl_sync(0xFFFFFFFFu, *abort_flag, 0) != 0) {
            break;                                     // spare warps
        }
    }

    // The leader lets the loads of both CTAs (they are counted on its barriers) and its MMAs finish
    // before either CTA gives up shared memory or TMEM; on the normal path these return at once.
    if (tid == 0) {
        for (uint32_t s = 0; s < (uint32_t)ns && s < it; ++s) {
            const uint32_t last = s + (it - 1 - s) / ns * ns;
            if (rank == 0) drain_phase(bar_full + 8 * s, (last / ns) & 1);
            if ((raw_used >> s) & 1u) drain_phase(bar_raw + 8 * s, ((raw_bits >> s) & 1u) ^ 1u);     // row pieces land on each CTA's own barrier
        }
    }
    if (rank == 0 && tid == 32) {
        ptx::mma_commit_pair(bar_drain, 1);
        drain_phase(bar_drain, 0);
    }
    // the peer cannot watch the leader's barriers: after a wait gave up it lets its last loads land for 2 ms
    if (rank == 1 && (tid == 0 || tid == 64) && *abort_flag)
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();          // no remote arrive, remote byte count or MMA of the pair is still under way
    if (warp == 1) ptx::tmem_dealloc_pair(tmem_base, 512);
}

// Standard normals of the matrices' P slots: one 16-byte store (8 bf16) per thread and pass.
__global__ void generate_p_kernel(const MatDesc* __restrict__ descs, int mat_begin, StepParams sp)
{
    const MatDesc* dp = descs + mat_begin + blockIdx.y;
    if (__ldg(&dp->path) != PATH_TENSOR) return;
    const int m_pad = __ldg(&dp->m_pad);
    const uint32_t matrix_id = (uint32_t)__ldg(&dp->matrix_id);
    uint4* out = static_cast<uint4*>(dp->pstage);
    const bool split = __ldg(&dp->split) != 0;
    const int chunks_per_row = (split ? 2 : 1) * (m_pad / 8);
    const int total = sp.rank_pad * chunks_per_row;
    const float* __restrict__ ext_p = dp->ext_p;
    const int m = __ldg(&dp->m);
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < total; c += gridDim.x * blockDim.x) {
        const int row = c / chunks_per_row, ch = c - row * chunks_per_row;
        out[c] = split ? p_vector<true>(ext_p, m, row, ch, matrix_id, sp, m_pad / 8)
                       : p_vector<false>(ext_p, m, row, ch, matrix_id, sp);
    }
}

}  // namespace

// G with an odd row pitch -> copy with the pitch rounded up to 8 elements (TMA needs 16-byte rows).
// One 16-byte store per thread and pass.  A source row starts `mis` bytes (even, the same for the whole
// row) past a 16-byte boundary of the array, so the eight elements of a store lie in two aligned
// 16-byte words: both are loaded (the second is the neighbouring thread's first) and the result is cut
// out with funnel shifts.  The padding columns are written as zero; the last vectors of the array, whose
// second word would reach past its end, are gathered element by element.
__global__ void repitch_kernel(const MatDesc* __restrict__ descs, int first)
{
    const MatDesc* dp = descs + first + blockIdx.y;
    uint4* dst = static_cast<uint4*>(dp->gpad);
    if (!dst) return;
    const unsigned short* __restrict__ src = static_cast<const unsigned short*>(dp->G);
    const char* __restrict__ src_b = static_cast<const char*>(dp->G);
    const int rows = __ldg(&dp->rows), cols = __ldg(&dp->cols), vecs = __ldg(&dp->g_pitch) / 8;
    const int64_t total_bytes = (int64_t)rows * cols * 2;
    for (int row = blockIdx.x; row < rows; row += gridDim.x) {
        const int64_t rb = (int64_t)row * cols * 2;
        const uint32_t mis = (uint32_t)(rb & 15), wsel = mis >> 2, sh = (mis & 2u) * 8u;
        for (int v = threadIdx.x; v < vecs; v += blockDim.x) {
            const int c = 8 * v;
            const int64_t a = rb - mis + 16 * (int64_t)v;
            uint32_t o[4];
            if (a + 32 <= total_bytes) {
                const uint4 lo = __ldg(reinterpret_cast<const uint4*>(src_b + a));
                const uint4 hi = __ldg(reinterpret_cast<const uint4*>(src_b + a + 16));
                const uint32_t w[8] = { lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w };
                switch (wsel) {          // uniform over the row
                case 0:
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[k] = __funnelshift_r(w[k], w[k + 1], sh);
                    break;
                case 1:
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[k] = __funnelshift_r(w[k + 1], w[k + 2], sh);
                    break;
                case 2:
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[k] = __funnelshift_r(w[k + 2], w[k + 3], sh);
                    break;
                default:
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[k] = __funnelshift_r(w[k + 3], w[k + 4], sh);
                    break;
                }
                if (c + 8 > cols) {      // the row ends inside this vector: what follows belongs to the next row
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (c + 2 * k >= cols) o[k] = 0u;
                        else if (c + 2 * k + 1 >= cols) o[k] &= 0xFFFFu;
                    }
                }
            } else {
                const unsigned short* __restrict__ in = src + (int64_t)row * cols;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t e0 = c + 2 * k < cols ? (uint32_t)__ldg(in + c + 2 * k) : 0u;
                    const uint32_t e1 = c + 2 * k + 1 < cols ? (uint32_t)__ldg(in + c + 2 * k + 1) : 0u;
                    o[k] = e0 | (e1 << 16);
                }
            }
            dst[(int64_t)row * vecs + v] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// fp32 gradient -> its bfloat16 high and low parts, [hi; lo] along the projected side, each part m_pad long
// (zero beyond m), for the three-segment contraction of the pair kernel; and the squared column norms of the
// gradient in fp32, which the tiles of the two parts cannot give (the cross term is missing there).
//   wide: a thread owns a column of one of four row slabs (coalesced over the 256 columns of a block); one
//         slice of norms per slab, summed by finalize_kernel.  tall: a warp owns a stored row (= channel).
__global__ void __launch_bounds__(256) split_kernel(const MatDesc* __restrict__ descs, int first)
{
    const MatDesc* dp = descs + first + blockIdx.y;
    if (__ldg(&dp->split) == 0) return;
    const float* __restrict__ G = static_cast<const float*>(dp->G);
    __nv_bfloat16* __restrict__ out = static_cast<__nv_bfloat16*>(dp->gpad);
    float* __restrict__ g2 = dp->g2;
    const int rows = __ldg(&dp->rows), cols = __ldg(&dp->cols), n = __ldg(&dp->n);
    const int m_pad = __ldg(&dp->m_pad);
    const int64_t pitch = __ldg(&dp->g_pitch);
    if (__ldg(&dp->tall) == 0) {
        const int ctiles = (cols + 255) / 256, rows_per = m_pad / 4;
        for (int u = blockIdx.x; u < 4 * ctiles; u += gridDim.x) {
            const int ct = u % ctiles, slab = u / ctiles, j = ct * 256 + (int)threadIdx.x;
            if (j >= cols) continue;
            float acc = 0.f;
            for (int i = slab * rows_per; i < (slab + 1) * rows_per; ++i) {
                const float g = i < rows ? __ldg(G + (int64_t)i * cols + j) : 0.f;
                const __nv_bfloat16 hi = __float2bfloat16_rn(g);
                out[(int64_t)i * pitch + j] = hi;
                out[(int64_t)(m_pad + i) * pitch + j] = __float2bfloat16_rn(g - __bfloat162float(hi));
                acc = fmaf(g, g, acc);
            }
            g2[(int64_t)slab * n + j] = acc;
        }
    } else {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int row = blockIdx.x * 8 + warp; row < rows; row += gridDim.x * 8) {
            float acc = 0.f;
            for (int c = lane; c < m_pad; c += 32) {
                const float g = c < cols ? __ldg(G + (int64_t)row * cols + c) : 0.f;
                const __nv_bfloat16 hi = __float2bfloat16_rn(g);
                out[(int64_t)row * pitch + c] = hi;
                out[(int64_t)row * pitch + m_pad + c] = __float2bfloat16_rn(g - __bfloat162float(hi));
                acc = fmaf(g, g, acc);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
            if (lane == 0) g2[row] = acc;
        }
    }
}

void launch_split(const MatDesc* d_descs, int first, int count, cudaStream_t stream)
{
    if (count <= 0) return;
    const dim3 grid(592, (unsigned)count);
    split_kernel<<<grid, 256, 0, stream>>>(d_descs, first);
}

void launch_repitch(const MatDesc* d_descs, int first, int count, cudaStream_t stream)
{
    if (count <= 0) return;
    const dim3 grid(592, (unsigned)count);
    repitch_kernel<<<grid, 256, 0, stream>>>(d_descs, first);
}

// One thread waits, with the bound every wait of the tensor kernel has, on an mbarrier that nothing
// arrives on.  The wait gives up, sets the status word and the block's flag; a second wait returns at
// once because the flag is set.  The kernel then ends normally: the context stays usable.
__global__ void bounded_wait_selftest_kernel(int32_t* status)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int flag;
    const uint32_t bar_addr = ptx::smem_addr(&bar);
    if (threadIdx.x == 0) {
        ptx::mbar_init(bar_addr, 1);
        flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool first = wait_phase(bar_addr, 0, &flag, status);
        const bool second = wait_phase(bar_addr, 0, &flag, status);
        if (first || second) atomicExch(status, STATUS_OK);   // a wait that "succeeded" here would be a defect: report no timeout
    }
}

void launch_bounded_wait_selftest(int32_t* d_status, cudaStream_t stream)
{
    bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(d_status);
}

void launch_generate_p(const MatDesc* d_descs, int mat_begin, int mat_end, const StepParams& sp, cudaStream_t stream)
{
    if (mat_end <= mat_begin) return;
    const dim3 grid(64, (unsigned)(mat_end - mat_begin));
    generate_p_kernel<<<grid, 256, 0, stream>>>(d_descs, mat_begin, sp);
}

void launch_project_tensor(const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                           const StepParams& sp, const TcTiling& tl, const GenArgs& gen, TcLaunchState& state,
                           int sm_count, int32_t* d_status, cudaStream_t stream)
{
    const int tiles = tile_end - tile_begin;
    if (tiles <= 0) return;
    // the shared-memory opt-in is a per-device attribute of the kernels: set once per context
    // the instantiation of the pair kernel for this context: re-aligned tiles, fp32 split, bfloat16 moments
    typedef void (*PairKernel)(const MatDesc*, const int*, int, int, int, StepParams, TcTiling, GenArgs, int32_t*);
    static const PairKernel pair_kernels[3][2] = {
        { project_pair_kernel<false, false, false>, project_pair_kernel<false, false, true> },
        { project_pair_kernel<true, false, false>, project_pair_kernel<true, false, true> },
        { project_pair_kernel<false, true, false>, project_pair_kernel<false, true, true> },
    };
    const PairKernel pair_kernel = pair_kernels[tl.split ? 2 : (tl.raw ? 1 : 0)][sp.state_bf16 ? 1 : 0];
    if (!state.attr_set) {
        cudaFuncSetAttribute(project_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_MAX_SMEM);
        cudaFuncSetAttribute(pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_MAX_SMEM);
        state.attr_set = true;
    }
    if (tl.pair) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(sm_count / 2 * 2);
        cfg.blockDim = dim3(P2_THREADS);
        cfg.dynamicSmemBytes = tl.smem_bytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        // the tile loop is persistent: launch exactly as many pairs as can be resident at once
        // (a pair sits in one GPC, so this can be fewer than half the SMs)
        if (state.max_pairs == 0) {
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, pair_kernel, &cfg) != cudaSuccess || clusters < 1) {
                cudaGetLastError();
                clusters = sm_count / 2;
            }
            state.max_pairs = clusters;
        }
        int pairs = state.max_pairs;
        if (tiles < pairs) pairs = tiles;
        cfg.gridDim = dim3(2 * pairs);
        cudaLaunchKernelEx(&cfg, pair_kernel, d_descs, d_prefix, n_mat, tile_begin, tile_end, sp, tl, gen, d_status);
        return;
    }
    const int grid = tiles < sm_count ? tiles : sm_count;
    project_tensor_kernel<<<grid, TC_THREADS, tl.smem_bytes, stream>>>(d_descs, d_prefix, n_mat, tile_begin, tile_end,
                                                                        sp, tl, d_status);
}

}  // namespace apollo
