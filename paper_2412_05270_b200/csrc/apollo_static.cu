// apollo_mini_step_static: one rank-1 (APOLLO-Mini style) step for a single matrix that
// allocates nothing.  Everything the regular step keeps in the caller's workspace apart
// from the optimizer state -- the matrix descriptor, the tile tables, the per-slice
// partial sums of the projection, the scales and the limiter scalars -- lives in one
// fixed-size array in device global memory that is part of the library image.  The
// kernels are the library's ordinary streaming-projection, finalize and update kernels,
// pointed at that array.
#include "../../include/apollo.h"

#include <cmath>
#include <mutex>

#include "apollo_internal.h"
#include "kernels.h"

using namespace apollo;

namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the
// process exits.  In host code `g_static_scratch` is only a handle for
// cudaGetSymbolAddress; it is not a device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[APOLLO_STATIC_SCRATCH_BYTES];

constexpr size_t OFF_DESC = 0;        // MatDesc
constexpr size_t OFF_PREFIX_P = 256;  // 2 ints: tile prefix of the projection
constexpr size_t OFF_PREFIX_U = 512;  // 2 ints: tile prefix of the update
constexpr size_t OFF_SCAL = 768;      // 4 floats: limiter outputs of the call
constexpr size_t OFF_ARRAYS = 1024;   // scales, then partial sums

constexpr int MAX_DEVICES = 64;
std::mutex g_mutex;
unsigned char* g_device_ptr[MAX_DEVICES];   // device address of the scratch, per device
int g_sm_count[MAX_DEVICES];
bool g_ready[MAX_DEVICES];

// Writes the descriptor and the two tile tables into the scratch (device code may name
// the array directly).
__global__ void static_setup_kernel(MatDesc d, int proj_tiles, int update_tiles)
{
    *reinterpret_cast<MatDesc*>(g_static_scratch + OFF_DESC) = d;
    int* pp = reinterpret_cast<int*>(g_static_scratch + OFF_PREFIX_P);
    int* pu = reinterpret_cast<int*>(g_static_scratch + OFF_PREFIX_U);
    pp[0] = 0; pp[1] = proj_tiles;
    pu[0] = 0; pu[1] = update_tiles;
    float* scal = reinterpret_cast<float*>(g_static_scratch + OFF_SCAL);
    scal[0] = 0.f; scal[1] = 0.f; scal[2] = 0.f; scal[3] = 0.f;   // nothing of an earlier call survives
}

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" int apollo_mini_step_static(void* d_W, const void* d_G, int64_t rows, int64_t cols,
                                       float* d_M, float* d_V, float* d_prev_norm,
                                       const apollo_config* cfg, uint32_t matrix, int64_t t,
                                       float lr, float wd, void* cuda_stream)
{
    if (!d_W || !d_G || !d_M || !d_V || !d_prev_norm || !cfg) return APOLLO_ERR_INVALID_ARG;
    if (cfg->rank != 1) return APOLLO_ERR_RANK;
    if (cfg->mode != APOLLO_SCALE_CHANNEL && cfg->mode != APOLLO_SCALE_TENSOR) return APOLLO_ERR_INVALID_ARG;
    if (cfg->dtype != APOLLO_DT_F32 && cfg->dtype != APOLLO_DT_BF16) return APOLLO_ERR_INVALID_ARG;
    if (cfg->T < 1 || t < 0 || !std::isfinite(lr) || !std::isfinite(wd)) return APOLLO_ERR_INVALID_ARG;
    if (!std::isfinite(cfg->alpha) || !std::isfinite(cfg->gamma) || !std::isfinite(cfg->eps) || cfg->eps < 0.f ||
        !(cfg->beta1 >= 0.f && cfg->beta1 <= 1.f) || !(cfg->beta2 >= 0.f && cfg->beta2 <= 1.f))
        return APOLLO_ERR_INVALID_ARG;
    if (cfg->bias_correction != 0 && cfg->bias_correction != 1) return APOLLO_ERR_INVALID_ARG;
    if (cfg->bias_correction && (cfg->beta1 >= 1.f || cfg->beta2 >= 1.f)) return APOLLO_ERR_INVALID_ARG;
    // d_M and d_V are n floats: a caller that asks for two-byte moments would be overrun
    if (cfg->flags & APOLLO_FLAG_BF16_STATES) return APOLLO_ERR_INVALID_ARG;
    if (rows < 1 || cols < 1 || rows > INT32_MAX || cols > INT32_MAX) return APOLLO_ERR_SHAPE;
    if (((uintptr_t)d_W % 16) || ((uintptr_t)d_G % 16) || ((uintptr_t)d_M % 16) || ((uintptr_t)d_V % 16) ||
        ((uintptr_t)d_prev_norm % 4))
        return APOLLO_ERR_ALIGN;

    MatDesc d{};
    d.rows = (int32_t)rows; d.cols = (int32_t)cols;
    d.tall = rows > cols;
    d.m = (int32_t)(d.tall ? cols : rows);
    d.n = (int32_t)(d.tall ? rows : cols);
    d.ns = d.n;
    d.path = PATH_STREAM;
    d.matrix_id = (int32_t)matrix;
    if (!d.tall) {
        d.tiles_n = (d.cols + STREAM_COLS - 1) / STREAM_COLS;
        d.tiles_k = (d.rows + STREAM_ROWS - 1) / STREAM_ROWS;
        d.slices = d.tiles_k;
    } else {
        d.tiles_n = (d.rows + STREAM_TALL_ROWS - 1) / STREAM_TALL_ROWS;
        d.tiles_k = 1;
        d.slices = 1;
    }
    const int64_t proj_tiles = (int64_t)d.tiles_n * d.tiles_k;
    const int64_t update_tiles = update_tile_count(rows, cols, d.tall != 0);
    d.upd_super = update_super_rows(rows, cols, d.tall != 0) ? 1 : 0;
    if (cols % 8 == 0 || d.upd_super) {
        const UpdateTiling ut = update_tiling((int)(d.upd_super ? 8 * cols : cols));
        d.upd_chunks = ut.chunks; d.upd_width = ut.width; d.upd_groups = ut.groups;
    }
    const size_t bytes_s = align256(sizeof(float) * (size_t)d.n);
    const size_t bytes_part = align256(sizeof(float) * 2 * (size_t)d.slices * (size_t)d.n);
    if (OFF_ARRAYS + bytes_s + bytes_part > (size_t)APOLLO_STATIC_SCRATCH_BYTES || proj_tiles > INT32_MAX ||
        update_tiles > INT32_MAX)
        return APOLLO_ERR_TOO_LARGE;

    // once per device, with that device current: the device address of the scratch
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return APOLLO_ERR_CUDA; }
    if (device < 0 || device >= MAX_DEVICES) return APOLLO_ERR_UNSUPPORTED;
    unsigned char* base = nullptr;
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_ready[device]) {
            int major = 0, sms = 0;
            void* ptr = nullptr;
            if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
                cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
                cudaGetLastError();
                return APOLLO_ERR_CUDA;
            }
            if (major != 10) return APOLLO_ERR_UNSUPPORTED;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
                cudaGetLastError();
                return APOLLO_ERR_CUDA;
            }
            g_device_ptr[device] = static_cast<unsigned char*>(ptr);
            g_sm_count[device] = sms;
            g_ready[device] = true;
        }
        base = g_device_ptr[device];
        sm_count = g_sm_count[device];
    }

    d.W = d_W; d.G = d_G; d.dW = nullptr;
    d.M = d_M; d.V = d_V; d.prev = d_prev_norm;
    d.scal = reinterpret_cast<float*>(base + OFF_SCAL);
    d.s = reinterpret_cast<float*>(base + OFF_ARRAYS);
    d.part = reinterpret_cast<float*>(base + OFF_ARRAYS + bytes_s);
    d.g2 = d.part;   // unused by the streaming path
    d.g2_slices = 0;
    d.ext_p = nullptr;
    d.r_scale = 1.0f;

    StepParams sp;
    sp.key0 = (uint32_t)(cfg->seed & 0xFFFFFFFFull);
    sp.key1 = (uint32_t)(cfg->seed >> 32);
    fill_round_keys(sp);
    sp.state_bf16 = 0;
    sp.epoch = (uint32_t)(t / cfg->T);
    sp.rank = 1; sp.rank_pad = 1; sp.mode = cfg->mode;
    sp.inv_sqrt_r = 1.0f;
    sp.lr = lr; sp.wd = wd; sp.alpha = cfg->alpha; sp.gamma = cfg->gamma;
    sp.beta1 = cfg->beta1; sp.beta2 = cfg->beta2; sp.eps = cfg->eps;
    sp.inv_bc1 = 1.f; sp.inv_bc2 = 1.f;
    if (cfg->bias_correction) {
        sp.inv_bc1 = (float)(1.0 / (1.0 - std::pow((double)cfg->beta1, (double)(t + 1))));
        sp.inv_bc2 = (float)(1.0 / (1.0 - std::pow((double)cfg->beta2, (double)(t + 1))));
    }

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const MatDesc* d_desc = reinterpret_cast<const MatDesc*>(base + OFF_DESC);
    static_setup_kernel<<<1, 1, 0, stream>>>(d, (int)proj_tiles, (int)update_tiles);
    launch_project_stream(cfg->dtype, d_desc, reinterpret_cast<const int*>(base + OFF_PREFIX_P), 1,
                          0, (int)proj_tiles, sp, sm_count, nullptr, stream);
    launch_finalize(d_desc, 0, 1, sp, nullptr, stream);
    launch_update(cfg->dtype, d_desc, reinterpret_cast<const int*>(base + OFF_PREFIX_U), 1, 0, (int)update_tiles,
                  sp, sm_count, nullptr, stream);
    return cudaGetLastError() == cudaSuccess ? APOLLO_OK : APOLLO_ERR_CUDA;
}
