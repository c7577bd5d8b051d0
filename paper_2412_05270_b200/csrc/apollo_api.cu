// Host side of libapollo: validation, workspace planning, descriptor tables and the
// launch sequence of one step (Algorithm 1): projection pass -> finalize -> update pass.
#include "../../include/apollo.h"

#include <nvtx3/nvToolsExt.h>

#include <cmath>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "apollo_internal.h"
#include "kernels.h"

using namespace apollo;

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

// An NVTX range on the calling thread, closed at the latest when the object goes out of scope.
struct NvtxRange {
    bool open;
    explicit NvtxRange(const char* name) : open(true) { nvtxRangePushA(name); }
    void close() { if (open) { nvtxRangePop(); open = false; } }
    ~NvtxRange() { close(); }
};

struct MatPlan {
    int32_t rows, cols, m, n, tall, path, slices, g2_slices, tiles_n, tiles_k, raw, split, g_pitch;
    int64_t proj_tiles, update_tiles;
    size_t off_M, off_V, off_scal, off_s, off_part, off_g2, off_tmap, off_pstage, off_gpad, gpad_bytes;
};

struct StageGroup {   // matrices whose P share one filling of the P scratch by generate_p_kernel
    int mat_begin, mat_end, tile_begin, tile_end;
};

struct Plan {
    std::vector<MatPlan> mats;
    size_t off_status, off_descs, off_prefix[4], off_tmaps, off_stage, stage_bytes, zero_begin, zero_end, total;
    size_t off_tmats, off_counters, counter_bytes;
    bool any_repitch;
    int64_t tiles[4];   // stream, simt, tensor, update
    std::vector<StageGroup> groups;
    std::vector<std::pair<int, int>> rp_groups;   // matrix ranges whose padded gradient copies share the repitch buffer
    int tc_rank;                    // the rank the tensor path works with (rounded up to the MMA's granularity)
    TcTiling tc;                    // tiling and mode of the tensor-core projection
    std::vector<int32_t> tensor_mats;   // tensor ordinal -> matrix index
    std::vector<int32_t> tq_prefix;     // matrix index -> number of tensor-path matrices before it
};

int validate_config(const apollo_config* cfg)
{
    if (!cfg) return APOLLO_ERR_INVALID_ARG;
    if (cfg->rank < 1 || cfg->rank > APOLLO_MAX_RANK) return APOLLO_ERR_RANK;
    if (cfg->mode != APOLLO_SCALE_CHANNEL && cfg->mode != APOLLO_SCALE_TENSOR) return APOLLO_ERR_INVALID_ARG;
    if (cfg->dtype != APOLLO_DT_F32 && cfg->dtype != APOLLO_DT_BF16) return APOLLO_ERR_INVALID_ARG;
    if (cfg->T < 1) return APOLLO_ERR_INVALID_ARG;
    if (!std::isfinite(cfg->alpha) || !std::isfinite(cfg->gamma) || !std::isfinite(cfg->eps) || cfg->eps < 0.f)
        return APOLLO_ERR_INVALID_ARG;
    if (!(cfg->beta1 >= 0.f && cfg->beta1 <= 1.f) || !(cfg->beta2 >= 0.f && cfg->beta2 <= 1.f))
        return APOLLO_ERR_INVALID_ARG;
    if (cfg->bias_correction != 0 && cfg->bias_correction != 1) return APOLLO_ERR_INVALID_ARG;
    if (cfg->bias_correction && (cfg->beta1 >= 1.f || cfg->beta2 >= 1.f)) return APOLLO_ERR_INVALID_ARG;
    return APOLLO_OK;
}

int make_plan(const apollo_shape* shapes, int32_t n_mat, const apollo_config* cfg, const apollo_tuning* tuning,
              Plan& plan)
{
    if (!shapes || n_mat < 1) return APOLLO_ERR_INVALID_ARG;
    int rc = validate_config(cfg);
    if (rc != APOLLO_OK) return rc;
    plan.tc = TcTiling{};
    plan.tc_rank = cfg->rank;
    if (cfg->rank >= 16) {
        plan.tc_rank = tensor_path_padded_rank(cfg->rank);
        rc = tensor_path_configure(plan.tc_rank, cfg->flags, tuning, &plan.tc);
        if (rc != APOLLO_OK) return rc;
        // fp32 gradients reach the tensor cores as bfloat16 high and low parts (pair kernel with a P scratch)
        plan.tc.split = cfg->dtype == APOLLO_DT_F32 && plan.tc.pair && plan.tc.staged ? 1 : 0;
    }
    plan.mats.resize(n_mat);
    for (int t = 0; t < 4; ++t) plan.tiles[t] = 0;
    const int r = cfg->rank;
    for (int i = 0; i < n_mat; ++i) {
        const int64_t rows = shapes[i].rows, cols = shapes[i].cols;
        if (rows < 1 || cols < 1 || rows > INT32_MAX || cols > INT32_MAX) return APOLLO_ERR_SHAPE;
        MatPlan& p = plan.mats[i];
        p.rows = (int32_t)rows; p.cols = (int32_t)cols;
        p.tall = rows > cols;
        p.m = (int32_t)(p.tall ? cols : rows);
        p.n = (int32_t)(p.tall ? rows : cols);
        if (r > p.m) return APOLLO_ERR_RANK;
        p.g2_slices = 0;
        if (r == 1) {
            p.path = PATH_STREAM;
            if (!p.tall) {
                p.tiles_n = (p.cols + STREAM_COLS - 1) / STREAM_COLS;
                p.tiles_k = (p.rows + STREAM_ROWS - 1) / STREAM_ROWS;
                p.slices = p.tiles_k;
            } else {
                p.tiles_n = (p.rows + STREAM_TALL_ROWS - 1) / STREAM_TALL_ROWS;
                p.tiles_k = 1;
                p.slices = 1;
            }
        } else if (tensor_path_supports(p.rows, p.cols, r, cfg->dtype, plan.tc) && !(cfg->flags & APOLLO_FLAG_NO_TENSOR_CORES)) {
            p.path = PATH_TENSOR;
            // rows that start on no 16-byte boundary: re-aligned in shared memory where the pair kernel can, else a padded copy
            p.split = plan.tc.split;
            p.raw = !p.split && tensor_path_raw_ok(p.rows, p.cols, plan.tc) ? 1 : 0;
            if (p.raw) tensor_path_enable_raw(&plan.tc);
            tensor_path_tiling(p.rows, p.cols, plan.tc_rank, plan.tc, &p.tiles_n, &p.tiles_k, &p.slices, &p.g2_slices);
        } else {
            p.path = PATH_SIMT;
            p.tiles_n = (p.n + SIMT_BN - 1) / SIMT_BN;
            p.tiles_k = (r + SIMT_BR - 1) / SIMT_BR;
            p.slices = p.tiles_k;
            p.g2_slices = 1;
        }
        p.proj_tiles = (int64_t)p.tiles_n * p.tiles_k;
        p.update_tiles = update_tile_count(rows, cols, p.tall != 0);
        plan.tiles[p.path] += p.proj_tiles;
        plan.tiles[3] += p.update_tiles;
    }
    for (int t = 0; t < 4; ++t)
        if (plan.tiles[t] > (int64_t)INT32_MAX - 1) return APOLLO_ERR_SHAPE;

    size_t off = 0;
    plan.off_status = off; off += ALIGN;
    plan.off_descs = off; off = align_up(off + sizeof(MatDesc) * (size_t)n_mat);
    for (int t = 0; t < 4; ++t) { plan.off_prefix[t] = off; off = align_up(off + sizeof(int) * ((size_t)n_mat + 1)); }
    plan.off_tmaps = off; off = align_up(off + 256 * (size_t)n_mat);
    // tensor-path matrices in list order
    plan.tensor_mats.clear();
    plan.tq_prefix.assign((size_t)n_mat + 1, 0);
    for (int i = 0; i < n_mat; ++i) {
        plan.tq_prefix[i] = (int32_t)plan.tensor_mats.size();
        if (plan.mats[i].path == PATH_TENSOR) plan.tensor_mats.push_back(i);
    }
    plan.tq_prefix[n_mat] = (int32_t)plan.tensor_mats.size();
    plan.off_tmats = off; off = align_up(off + sizeof(int32_t) * (plan.tensor_mats.size() + 1));
    // generator counters of the pair kernel: ticket, then per matrix pieces written and tiles read
    plan.counter_bytes = align_up(sizeof(uint32_t) * (1 + 2 * (size_t)n_mat));
    plan.off_counters = off; off += plan.counter_bytes;
    // The P scratch.  kept: every matrix owns a slot.  gen: a ring of equal slots over the tensor ordinals.
    // Otherwise staging groups: consecutive matrices whose P fit the scratch together, filled group by group.
    plan.groups.clear();
    plan.stage_bytes = 0;
    if (plan.tc.gen) {
        // A list whose projections all fit the scratch is served better by the separate generator kernel, once
        // per step and with the whole chip (44 M normals of the 350M list: 40 us), than by the spare warps of
        // the pair kernel, which then sit on the critical path (such lists have few tiles per matrix).
        size_t all = 0;
        for (int i : plan.tensor_mats)
            all += align_up(tensor_path_stage_bytes(plan.mats[i].rows, plan.mats[i].cols, plan.tc_rank, plan.mats[i].split != 0));
        if (plan.tc.gen == 1 && all <= (size_t)plan.tc.scratch_bytes) plan.tc.gen = 0;
    }
    if (plan.tc.gen && !plan.tensor_mats.empty()) {
        size_t slot = 0;
        for (int i : plan.tensor_mats) {
            const size_t need = align_up(tensor_path_stage_bytes(plan.mats[i].rows, plan.mats[i].cols, plan.tc_rank, plan.mats[i].split != 0));
            if (need > slot) slot = need;
        }
        const int64_t ring_bytes = plan.tc.scratch_bytes < ((int64_t)32 << 20) ? plan.tc.scratch_bytes : ((int64_t)32 << 20);
        int64_t slots = ring_bytes / (int64_t)slot;      // a deeper ring gains nothing (32, 64 and 256 MB measured equal)
        if (slots < 2) slots = 2;
        if (slots > (int64_t)plan.tensor_mats.size()) slots = (int64_t)plan.tensor_mats.size();
        plan.tc.slots = (int32_t)slots;
        for (size_t q = 0; q < plan.tensor_mats.size(); ++q)
            plan.mats[plan.tensor_mats[q]].off_pstage = (q % (size_t)slots) * slot;
        plan.stage_bytes = (size_t)slots * slot;
        plan.groups.push_back(StageGroup{ 0, n_mat, 0, (int)plan.tiles[PATH_TENSOR] });
    } else {
        const size_t budget = plan.tc.keep ? (size_t)-1 : (size_t)plan.tc.scratch_bytes;
        StageGroup g = { 0, 0, 0, 0 };
        size_t used = 0;
        int tile_at = 0;
        for (int i = 0; i < n_mat; ++i) {
            MatPlan& p = plan.mats[i];
            const bool tensor = p.path == PATH_TENSOR;
            const size_t need = tensor && plan.tc.staged ? align_up(tensor_path_stage_bytes(p.rows, p.cols, plan.tc_rank, p.split != 0)) : 0;
            if (used > 0 && (used >= budget || need > budget - used)) {
                g.mat_end = i; g.tile_end = tile_at;
                plan.groups.push_back(g);
                g.mat_begin = i; g.tile_begin = tile_at;
                used = 0;
            }
            p.off_pstage = used;
            used += need;
            if (used > plan.stage_bytes) plan.stage_bytes = used;
            if (tensor) tile_at += (int)p.proj_tiles;
        }
        g.mat_end = n_mat; g.tile_end = tile_at;
        plan.groups.push_back(g);
    }
    plan.off_stage = off; off = align_up(off + plan.stage_bytes);
    // padded copies of the gradients whose row pitch TMA cannot take (cols not a multiple of 8)
    plan.any_repitch = false;
    plan.rp_groups.clear();
    {
        // consecutive matrices share the buffer until their copies would exceed the budget; then the next group
        // starts again at its beginning (each group is copied and projected before the next one is copied)
        const size_t budget = plan.tc.repitch_bytes > 0 ? (size_t)plan.tc.repitch_bytes : (size_t)-1;
        size_t used = 0, largest = 0;
        int begin = 0;
        for (int i = 0; i < n_mat; ++i) {
            MatPlan& p = plan.mats[i];
            p.gpad_bytes = 0;
            p.g_pitch = p.cols;
            if (p.path == PATH_TENSOR && p.split) {
                int pitch = 0;
                p.gpad_bytes = align_up(tensor_path_split_bytes(p.rows, p.cols, &pitch));
                p.g_pitch = pitch;
                plan.any_repitch = true;
            } else if (p.path == PATH_TENSOR && (p.cols % 8) != 0 && !p.raw) {
                p.g_pitch = (p.cols + 7) / 8 * 8;
                p.gpad_bytes = align_up((size_t)p.rows * (size_t)p.g_pitch * 2);
                plan.any_repitch = true;
            }
            if (used > 0 && p.gpad_bytes > 0 && (used >= budget || p.gpad_bytes > budget - used)) {
                plan.rp_groups.push_back({ begin, i });
                begin = i;
                used = 0;
            }
            p.off_gpad = off + used;
            used += p.gpad_bytes;
            if (used > largest) largest = used;
        }
        plan.rp_groups.push_back({ begin, n_mat });
        off = align_up(off + largest);
    }
    plan.zero_begin = off;
    for (int i = 0; i < n_mat; ++i) {
        MatPlan& p = plan.mats[i];
        const size_t state = ((cfg->flags & APOLLO_FLAG_BF16_STATES) ? 2 : sizeof(float)) * (size_t)state_elements(p.n, p.path == PATH_TENSOR ? plan.tc_rank : r, p.path == PATH_TENSOR);
        p.off_M = off; off = align_up(off + state);
        p.off_V = off; off = align_up(off + state);
        p.off_scal = off; off += ALIGN;     // scal[4] then prev at float index 8
    }
    plan.zero_end = off;
    for (int i = 0; i < n_mat; ++i) {
        MatPlan& p = plan.mats[i];
        p.off_s = off; off = align_up(off + sizeof(float) * (size_t)p.n);
        p.off_part = off; off = align_up(off + sizeof(float) * 2 * (size_t)p.slices * (size_t)p.n);
        p.off_g2 = off; off = align_up(off + sizeof(float) * (size_t)(p.g2_slices > 0 ? p.g2_slices : 1) * (size_t)p.n);
        p.off_tmap = plan.off_tmaps + 256 * (size_t)i;
    }
    plan.total = off;
    return APOLLO_OK;
}

}  // namespace

static thread_local cudaError_t g_last_cuda_error = cudaSuccess;

// Records a failing CUDA status for apollo_cuda_error_string(); returns true on success.
static bool cuda_ok(cudaError_t e)
{
    if (e != cudaSuccess) { g_last_cuda_error = e; cudaGetLastError(); return false; }
    return true;
}

// Pinned host staging of the descriptor table and the tensor maps: an upload from pageable memory would
// make cudaMemcpyAsync wait for the stream.  Two slots, each reused once the copy recorded in it is done.
struct UploadSlot {
    char* host;
    cudaEvent_t done;
    bool in_flight;
};

struct apollo_ctx {
    apollo_config cfg;
    int32_t n_mat;
    Plan plan;
    TcLaunchState tc_state;
    std::vector<char> h_maps;        // 2 x n_mat tensor maps of 128 bytes (G, the matrix's P slot)
    UploadSlot upload[2];
    int upload_next;
    std::vector<MatDesc> h_descs;
    std::vector<int> h_prefix[4];
    char* ws;
    MatDesc* d_descs;
    int* d_prefix[4];
    int32_t* d_status;
    std::vector<float*> delta;
    bool delta_on;
    bool first;
    bool imported;   // the moments came from apollo_state_import: the first step must not zero them
    bool descs_dirty;
    std::vector<int64_t> staged_epoch;   // per matrix: the epoch whose P its staging slot holds, -1 = none
    int64_t t;
    int device;
    int sm_count;
    int last_launches;
    bool timing_on;
    bool timing_ready;
    cudaEvent_t ev[APOLLO_TIMING_SLOTS][4];
};

extern "C" {

const char* apollo_cuda_error_string(void) { return cudaGetErrorString(g_last_cuda_error); }

const char* apollo_strerror(int code)
{
    switch (code) {
        case APOLLO_OK: return "ok";
        case APOLLO_ERR_INVALID_ARG: return "invalid argument";
        case APOLLO_ERR_SHAPE: return "unsupported shape";
        case APOLLO_ERR_RANK: return "rank out of range for a matrix";
        case APOLLO_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case APOLLO_ERR_WORKSPACE: return "workspace too small or misaligned";
        case APOLLO_ERR_CUDA: return "CUDA call failed";
        case APOLLO_ERR_TIMEOUT: return "bounded device-side wait expired";
        case APOLLO_ERR_UNSUPPORTED: return "device is not an sm_100 GPU";
        case APOLLO_ERR_TOO_LARGE: return "matrix exceeds the built-in scratch of apollo_mini_step_static";
        case APOLLO_ERR_INTERNAL: return "an index check inside a kernel failed (debug build)";
        default: return "unknown error";
    }
}

int apollo_workspace_bytes_tuned(const apollo_shape* shapes, int32_t n_matrices, const apollo_config* cfg,
                                 const apollo_tuning* tuning, size_t* out_bytes)
{
    if (!out_bytes) return APOLLO_ERR_INVALID_ARG;
    Plan plan;
    const int rc = make_plan(shapes, n_matrices, cfg, tuning, plan);
    if (rc != APOLLO_OK) return rc;
    *out_bytes = plan.total;
    return APOLLO_OK;
}

int apollo_workspace_bytes(const apollo_shape* shapes, int32_t n_matrices, const apollo_config* cfg,
                           size_t* out_bytes)
{
    return apollo_workspace_bytes_tuned(shapes, n_matrices, cfg, nullptr, out_bytes);
}

int apollo_create(apollo_ctx** out_ctx, const apollo_shape* shapes, int32_t n_matrices,
                  const apollo_config* cfg, void* d_workspace, size_t workspace_bytes)
{
    return apollo_create_tuned(out_ctx, shapes, n_matrices, cfg, nullptr, d_workspace, workspace_bytes);
}

int apollo_create_tuned(apollo_ctx** out_ctx, const apollo_shape* shapes, int32_t n_matrices,
                        const apollo_config* cfg, const apollo_tuning* tuning, void* d_workspace,
                        size_t workspace_bytes)
{
    if (!out_ctx) return APOLLO_ERR_INVALID_ARG;
    *out_ctx = nullptr;
    apollo_ctx* ctx = new (std::nothrow) apollo_ctx();
    if (!ctx) return APOLLO_ERR_INVALID_ARG;
    int rc = make_plan(shapes, n_matrices, cfg, tuning, ctx->plan);
    if (rc != APOLLO_OK) { delete ctx; return rc; }
    if (!d_workspace) { delete ctx; return APOLLO_ERR_INVALID_ARG; }
    if (((uintptr_t)d_workspace % ALIGN) != 0 || workspace_bytes < ctx->plan.total) { delete ctx; return APOLLO_ERR_WORKSPACE; }

    int device = 0, major = 0, sms = 0;
    if (cudaGetDevice(&device) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        cudaGetLastError();
        delete ctx; return APOLLO_ERR_CUDA;
    }
    if (major != 10) { delete ctx; return APOLLO_ERR_UNSUPPORTED; }

    ctx->cfg = *cfg;
    ctx->n_mat = n_matrices;
    ctx->ws = static_cast<char*>(d_workspace);
    ctx->device = device;
    ctx->sm_count = sms;
    ctx->d_status = reinterpret_cast<int32_t*>(ctx->ws + ctx->plan.off_status);
    ctx->d_descs = reinterpret_cast<MatDesc*>(ctx->ws + ctx->plan.off_descs);
    ctx->h_descs.resize(n_matrices);
    for (int t = 0; t < 4; ++t) {
        ctx->d_prefix[t] = reinterpret_cast<int*>(ctx->ws + ctx->plan.off_prefix[t]);
        ctx->h_prefix[t].assign(n_matrices + 1, 0);
    }
    for (int i = 0; i < n_matrices; ++i) {
        const MatPlan& p = ctx->plan.mats[i];
        MatDesc& d = ctx->h_descs[i];
        std::memset(&d, 0, sizeof(d));
        d.M = reinterpret_cast<float*>(ctx->ws + p.off_M);
        d.V = reinterpret_cast<float*>(ctx->ws + p.off_V);
        d.scal = reinterpret_cast<float*>(ctx->ws + p.off_scal);
        d.prev = d.scal + 8;
        d.s = reinterpret_cast<float*>(ctx->ws + p.off_s);
        d.part = reinterpret_cast<float*>(ctx->ws + p.off_part);
        d.g2 = reinterpret_cast<float*>(ctx->ws + p.off_g2);
        d.tmap = ctx->ws + p.off_tmap;
        d.tmap_p = ctx->ws + p.off_tmap + 128;
        d.pstage = ctx->ws + ctx->plan.off_stage + p.off_pstage;
        d.m_pad = (p.m + 63) / 64 * 64;
        d.gpad = p.gpad_bytes ? ctx->ws + p.off_gpad : nullptr;
        d.g_pitch = p.g_pitch;
        d.raw = p.raw;
        d.split = p.split;
        d.p_width = (p.split ? 2 : 1) * d.m_pad;
        d.upd_super = update_super_rows(p.rows, p.cols, p.tall != 0) ? 1 : 0;
        if (p.cols % 8 == 0 || d.upd_super) {
            const UpdateTiling ut = update_tiling(d.upd_super ? 8 * p.cols : p.cols);
            d.upd_chunks = ut.chunks; d.upd_width = ut.width; d.upd_groups = ut.groups;
        } else {
            d.upd_chunks = 0; d.upd_width = 0; d.upd_groups = 0;
        }
        d.ext_p = nullptr;
        d.r_scale = (float)(1.0 / std::sqrt((double)cfg->rank));
        d.rows = p.rows; d.cols = p.cols; d.m = p.m; d.n = p.n; d.tall = p.tall; d.path = p.path;
        d.ns = state_pitch(p.n, cfg->rank);
        d.state_tiled = p.path == PATH_TENSOR ? 1 : 0;
        d.slices = p.slices; d.g2_slices = p.g2_slices; d.matrix_id = i;
        d.tiles_n = p.tiles_n; d.tiles_k = p.tiles_k;
        for (int t = 0; t < 3; ++t)
            ctx->h_prefix[t][i + 1] = ctx->h_prefix[t][i] + (p.path == t ? (int)p.proj_tiles : 0);
        ctx->h_prefix[3][i + 1] = ctx->h_prefix[3][i] + (int)p.update_tiles;
    }
    ctx->tc_state = TcLaunchState{ false, 0 };
    ctx->h_maps.assign(256 * (size_t)n_matrices, 0);
    ctx->upload_next = 0;
    for (UploadSlot& u : ctx->upload) {
        u.host = nullptr; u.done = nullptr; u.in_flight = false;
        void* host = nullptr;
        if (cudaHostAlloc(&host, sizeof(MatDesc) * (size_t)n_matrices + 256 * (size_t)n_matrices, cudaHostAllocDefault) ==
                cudaSuccess &&
            cudaEventCreateWithFlags(&u.done, cudaEventDisableTiming) == cudaSuccess) {
            u.host = static_cast<char*>(host);
        } else {
            cudaGetLastError();          // no pinned memory to be had: uploads go from pageable memory
            if (host) cudaFreeHost(host);
            u.done = nullptr;
        }
    }
    ctx->delta.assign(n_matrices, nullptr);
    ctx->delta_on = false;
    ctx->first = true;
    ctx->imported = false;
    ctx->staged_epoch.assign((size_t)ctx->n_mat, -1);
    ctx->descs_dirty = true;
    ctx->t = 0;
    ctx->last_launches = 0;
    ctx->timing_on = false;
    ctx->timing_ready = false;
    *out_ctx = ctx;
    return APOLLO_OK;
}

int apollo_destroy(apollo_ctx* ctx)
{
    if (!ctx) return APOLLO_ERR_INVALID_ARG;
    if (ctx->timing_ready)
        for (int sl = 0; sl < APOLLO_TIMING_SLOTS; ++sl)
            for (int e = 0; e < 4; ++e) cudaEventDestroy(ctx->ev[sl][e]);
    for (UploadSlot& u : ctx->upload) {
        if (u.host) {
            if (u.in_flight) cudaEventSynchronize(u.done);
            cudaEventDestroy(u.done);
            cudaFreeHost(u.host);
        }
    }
    delete ctx;
    return APOLLO_OK;
}

int apollo_step_count(const apollo_ctx* ctx, int64_t* out)
{
    if (!ctx || !out) return APOLLO_ERR_INVALID_ARG;
    *out = ctx->t;
    return APOLLO_OK;
}

int apollo_set_delta_out(apollo_ctx* ctx, float* const* d_dW)
{
    if (!ctx) return APOLLO_ERR_INVALID_ARG;
    if (d_dW) {
        for (int i = 0; i < ctx->n_mat; ++i)
            if ((uintptr_t)d_dW[i] % 16) return APOLLO_ERR_ALIGN;   // a null entry skips that matrix
        for (int i = 0; i < ctx->n_mat; ++i) ctx->delta[i] = d_dW[i];
        ctx->delta_on = true;
    } else {
        ctx->delta.assign(ctx->n_mat, nullptr);
        ctx->delta_on = false;
    }
    ctx->descs_dirty = true;
    return APOLLO_OK;
}

// One step of matrices [first, first + count) at the current step counter; d_W and d_G hold
// `count` pointers.  `advance` closes the step (t <- t + 1).
static int step_range(apollo_ctx* ctx, int first, int count, void* const* d_W, const void* const* d_G, float lr,
                      float wd, bool advance, void* cuda_stream)
{
    if (!ctx || !d_W || !d_G) return APOLLO_ERR_INVALID_ARG;
    if (first < 0 || count < 1 || first + count > ctx->n_mat) return APOLLO_ERR_INVALID_ARG;
    if (!std::isfinite(lr) || !std::isfinite(wd)) return APOLLO_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        if (!d_W[i] || !d_G[i]) return APOLLO_ERR_INVALID_ARG;
        if (((uintptr_t)d_W[i] % 16) || ((uintptr_t)d_G[i] % 16)) return APOLLO_ERR_ALIGN;
    }
    const int last = first + count;
    const bool whole = count == ctx->n_mat;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const apollo_config& cfg = ctx->cfg;
    const Plan& plan = ctx->plan;

    if (ctx->first) {
        if (cudaMemsetAsync(ctx->ws + plan.off_status, 0, ALIGN, stream) != cudaSuccess) return APOLLO_ERR_CUDA;
        if (!ctx->imported &&
            cudaMemsetAsync(ctx->ws + plan.zero_begin, 0, plan.zero_end - plan.zero_begin, stream) != cudaSuccess)
            return APOLLO_ERR_CUDA;
        for (int t = 0; t < 4; ++t)
            if (cudaMemcpyAsync(ctx->d_prefix[t], ctx->h_prefix[t].data(), sizeof(int) * (ctx->n_mat + 1),
                                cudaMemcpyHostToDevice, stream) != cudaSuccess)
                return APOLLO_ERR_CUDA;
        if (!plan.tensor_mats.empty() &&
            cudaMemcpyAsync(ctx->ws + plan.off_tmats, plan.tensor_mats.data(), sizeof(int32_t) * plan.tensor_mats.size(),
                            cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return APOLLO_ERR_CUDA;
    }
    // A tensor map depends on the matrix's G address alone (the map of its P slot never changes): matrices
    // whose G moved get a new one; the whole table travels with the descriptors when anything changed.
    bool changed = ctx->descs_dirty;
    for (int i = first; i < last; ++i) {
        MatDesc& d = ctx->h_descs[i];
        const bool g_moved = d.G != d_G[i - first];
        if (d.W != d_W[i - first] || g_moved || d.dW != ctx->delta[i]) {
            d.W = d_W[i - first]; d.G = d_G[i - first]; d.dW = ctx->delta[i];
            changed = true;
        }
        if ((g_moved || ctx->first) && d.path == PATH_TENSOR) {
            const int rc = tensor_path_prepare(&d, 1, plan.tc_rank, plan.tc, ctx->h_maps.data() + 256 * (size_t)i);
            if (rc != APOLLO_OK) return rc;
        }
    }
    if (changed) {
        const size_t desc_bytes = sizeof(MatDesc) * (size_t)ctx->n_mat, map_bytes = 256 * (size_t)ctx->n_mat;
        const char* src_descs = reinterpret_cast<const char*>(ctx->h_descs.data());
        const char* src_maps = ctx->h_maps.data();
        UploadSlot& u = ctx->upload[ctx->upload_next];
        if (u.host) {
            if (u.in_flight && cudaEventSynchronize(u.done) != cudaSuccess) return APOLLO_ERR_CUDA;   // two uploads ago
            std::memcpy(u.host, src_descs, desc_bytes);
            std::memcpy(u.host + desc_bytes, src_maps, map_bytes);
            src_descs = u.host; src_maps = u.host + desc_bytes;
        }
        if (cudaMemcpyAsync(ctx->d_descs, src_descs, desc_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            cudaMemcpyAsync(ctx->ws + plan.off_tmaps, src_maps, map_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return APOLLO_ERR_CUDA;
        if (u.host) {
            if (cudaEventRecord(u.done, stream) != cudaSuccess) return APOLLO_ERR_CUDA;
            u.in_flight = true;
            ctx->upload_next ^= 1;
        }
        ctx->descs_dirty = false;
    }

    StepParams sp;
    sp.key0 = (uint32_t)(cfg.seed & 0xFFFFFFFFull);
    sp.key1 = (uint32_t)(cfg.seed >> 32);
    fill_round_keys(sp);
    sp.state_bf16 = (cfg.flags & APOLLO_FLAG_BF16_STATES) ? 1 : 0;
    sp.epoch = (uint32_t)(ctx->t / cfg.T);
    sp.rank = cfg.rank; sp.mode = cfg.mode;
    sp.rank_pad = plan.tc_rank;
    sp.inv_sqrt_r = (float)(1.0 / std::sqrt((double)cfg.rank));
    sp.lr = lr; sp.wd = wd; sp.alpha = cfg.alpha; sp.gamma = cfg.gamma;
    sp.beta1 = cfg.beta1; sp.beta2 = cfg.beta2; sp.eps = cfg.eps;
    sp.inv_bc1 = 1.f; sp.inv_bc2 = 1.f;
    if (cfg.bias_correction) {
        sp.inv_bc1 = (float)(1.0 / (1.0 - std::pow((double)cfg.beta1, (double)(ctx->t + 1))));
        sp.inv_bc2 = (float)(1.0 / (1.0 - std::pow((double)cfg.beta2, (double)(ctx->t + 1))));
    }

    // NVTX ranges around the three phases (host side of the launches): a timeline tool shows them, and
    // without one attached each call is a pointer test
    int launches = 0;
    cudaEvent_t* ev = (ctx->timing_on && whole) ? ctx->ev[ctx->t % APOLLO_TIMING_SLOTS] : nullptr;
    if (ev) cudaEventRecord(ev[0], stream);
    NvtxRange range_projection("apollo.projection");
    auto tiles_of = [&](int path, int a, int b, int& tb, int& te) {
        tb = ctx->h_prefix[path][a]; te = ctx->h_prefix[path][b];
        return te > tb;
    };
    int tb = 0, te = 0;
    if (tiles_of(PATH_STREAM, first, last, tb, te)) {
        launch_project_stream(cfg.dtype, ctx->d_descs, ctx->d_prefix[PATH_STREAM], ctx->n_mat, tb, te, sp,
                              ctx->sm_count, ctx->d_status, stream);
        ++launches;
    }
    if (tiles_of(PATH_SIMT, first, last, tb, te)) {
        launch_project_simt(cfg.dtype, ctx->d_descs, ctx->d_prefix[PATH_SIMT], ctx->n_mat, tb, te, sp, ctx->sm_count,
                            ctx->d_status, stream);
        ++launches;
    }
    // The padded copies of gradients with an unaligned row pitch share one buffer group by group (one group
    // when there are none): each group's part of the range is copied, then projected, before the next is copied.
    for (const std::pair<int, int>& rg : plan.rp_groups) {
        const int ra = rg.first > first ? rg.first : first;
        const int rb = rg.second < last ? rg.second : last;
        if (rb <= ra || !tiles_of(PATH_TENSOR, ra, rb, tb, te)) continue;
        if (plan.any_repitch) {
            bool any = false;
            for (int i = ra; i < rb; ++i) any |= ctx->h_descs[i].gpad != nullptr;
            if (any) {
                if (plan.tc.split) launch_split(ctx->d_descs, ra, rb - ra, stream);
                else launch_repitch(ctx->d_descs, ra, rb - ra, stream);
                ++launches;
            }
        }
        const TcTiling& tc = plan.tc;
        GenArgs gen = {};
        if (tc.gen) {
            // one launch over the range: spare warps of the kernel regenerate every matrix's P from the seed,
            // a few matrices ahead of the tiles that read it, through the ring of slots in the scratch
            uint32_t* counters = reinterpret_cast<uint32_t*>(ctx->ws + plan.off_counters);
            if (cudaMemsetAsync(counters, 0, plan.counter_bytes, stream) != cudaSuccess) return APOLLO_ERR_CUDA;
            gen.mats = reinterpret_cast<const int32_t*>(ctx->ws + plan.off_tmats);
            gen.q_begin = plan.tq_prefix[ra]; gen.q_end = plan.tq_prefix[rb];
            gen.ticket = counters; gen.gen_done = counters + 1; gen.use_done = counters + 1 + ctx->n_mat;
            launch_project_tensor(ctx->d_descs, ctx->d_prefix[PATH_TENSOR], ctx->n_mat, tb, te, sp, tc, gen,
                                  ctx->tc_state, ctx->sm_count, ctx->d_status, stream);
            ++launches;
        } else {
            for (const StageGroup& g : plan.groups) {
                // the part of this staging group inside the range
                const int mb = g.mat_begin > ra ? g.mat_begin : ra;
                const int me = g.mat_end < rb ? g.mat_end : rb;
                if (me <= mb || !tiles_of(PATH_TENSOR, mb, me, tb, te)) continue;
                if (tc.staged) {
                    // P changes only with the epoch (every T steps).  When every matrix keeps its own slot
                    // (APOLLO_FLAG_KEEP_P), a slot filled in this epoch is read again instead of being regenerated.
                    // A projection supplied by the caller is converted every step: its buffer may have been rewritten.
                    int lo = mb, hi = me;
                    if (tc.keep) {
                        auto fresh = [&](int i) {
                            const MatDesc& d = ctx->h_descs[i];
                            return d.path != PATH_TENSOR || (!d.ext_p && ctx->staged_epoch[i] == (int64_t)sp.epoch);
                        };
                        while (lo < hi && fresh(lo)) ++lo;
                        while (hi > lo && fresh(hi - 1)) --hi;
                        for (int i = lo; i < hi; ++i) ctx->staged_epoch[i] = (int64_t)sp.epoch;
                    }
                    if (hi > lo) {
                        launch_generate_p(ctx->d_descs, lo, hi, sp, stream);
                        ++launches;
                    }
                }
                launch_project_tensor(ctx->d_descs, ctx->d_prefix[PATH_TENSOR], ctx->n_mat, tb, te, sp, tc, gen,
                                      ctx->tc_state, ctx->sm_count, ctx->d_status, stream);
                ++launches;
            }
        }
    }
    range_projection.close();
    if (ev) cudaEventRecord(ev[1], stream);
    NvtxRange range_finalize("apollo.finalize");
    launch_finalize(ctx->d_descs, first, count, sp, ctx->d_status, stream);
    ++launches;
    range_finalize.close();
    if (ev) cudaEventRecord(ev[2], stream);
    NvtxRange range_update("apollo.update");
    tiles_of(3, first, last, tb, te);
    launch_update(cfg.dtype, ctx->d_descs, ctx->d_prefix[3], ctx->n_mat, tb, te, sp, ctx->sm_count, ctx->d_status, stream);
    ++launches;
    range_update.close();
    if (ev) cudaEventRecord(ev[3], stream);
    if (!cuda_ok(cudaGetLastError())) return APOLLO_ERR_CUDA;
    ctx->first = false;
    if (advance) ctx->t += 1;
    ctx->last_launches = launches;
    return APOLLO_OK;
}

int apollo_step(apollo_ctx* ctx, void* const* d_W, const void* const* d_G, float lr, float wd,
                void* cuda_stream)
{
    if (!ctx) return APOLLO_ERR_INVALID_ARG;
    return step_range(ctx, 0, ctx->n_mat, d_W, d_G, lr, wd, true, cuda_stream);
}

int apollo_step_range(apollo_ctx* ctx, int32_t first, int32_t count, void* const* d_W, const void* const* d_G,
                      float lr, float wd, int32_t close_step, void* cuda_stream)
{
    return step_range(ctx, first, count, d_W, d_G, lr, wd, close_step != 0, cuda_stream);
}

int apollo_get_scales(apollo_ctx* ctx, int32_t matrix, float* d_out, void* cuda_stream)
{
    if (!ctx || !d_out || matrix < 0 || matrix >= ctx->n_mat) return APOLLO_ERR_INVALID_ARG;
    const MatDesc& d = ctx->h_descs[matrix];
    return cudaMemcpyAsync(d_out, d.s, sizeof(float) * d.n, cudaMemcpyDeviceToDevice,
                           static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? APOLLO_OK : APOLLO_ERR_CUDA;
}

int apollo_get_limiter(apollo_ctx* ctx, int32_t matrix, float* d_out, void* cuda_stream)
{
    if (!ctx || !d_out || matrix < 0 || matrix >= ctx->n_mat) return APOLLO_ERR_INVALID_ARG;
    const MatDesc& d = ctx->h_descs[matrix];
    return cudaMemcpyAsync(d_out, d.scal, sizeof(float) * 4, cudaMemcpyDeviceToDevice,
                           static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? APOLLO_OK : APOLLO_ERR_CUDA;
}

int apollo_get_state(apollo_ctx* ctx, int32_t matrix, float* d_M, float* d_V, void* cuda_stream)
{
    if (!ctx || !d_M || !d_V || matrix < 0 || matrix >= ctx->n_mat) return APOLLO_ERR_INVALID_ARG;
    const MatDesc& d = ctx->h_descs[matrix];
    const size_t r = (size_t)ctx->cfg.rank, n = (size_t)d.n, ns = (size_t)d.ns;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool bf16 = (ctx->cfg.flags & APOLLO_FLAG_BF16_STATES) != 0;
    if (bf16 || d.state_tiled) {
        // the caller gets dense fp32 rows whatever the library's layout and storage type
        launch_state_copy(d.M, d_M, (int)r, ctx->plan.tc_rank, d.n, d.ns, d.state_tiled != 0, bf16 ? 2 : 4, 4, true, stream);
        launch_state_copy(d.V, d_V, (int)r, ctx->plan.tc_rank, d.n, d.ns, d.state_tiled != 0, bf16 ? 2 : 4, 4, true, stream);
        return cuda_ok(cudaGetLastError()) ? APOLLO_OK : APOLLO_ERR_CUDA;
    }
    // the library's rows have pitch ns; the caller gets them dense
    if (cudaMemcpy2DAsync(d_M, sizeof(float) * n, d.M, sizeof(float) * ns, sizeof(float) * n, r, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) return APOLLO_ERR_CUDA;
    if (cudaMemcpy2DAsync(d_V, sizeof(float) * n, d.V, sizeof(float) * ns, sizeof(float) * n, r, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) return APOLLO_ERR_CUDA;
    return APOLLO_OK;
}

int apollo_selftest_bounded_wait(apollo_ctx* ctx, void* cuda_stream)
{
    if (!ctx || ctx->first) return APOLLO_ERR_INVALID_ARG;   // the status word exists once a step has run
    launch_bounded_wait_selftest(ctx->d_status, static_cast<cudaStream_t>(cuda_stream));
    return cuda_ok(cudaGetLastError()) ? APOLLO_OK : APOLLO_ERR_CUDA;
}

int apollo_status(apollo_ctx* ctx, void* cuda_stream)
{
    if (!ctx) return APOLLO_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return APOLLO_ERR_CUDA;
    if (ctx->first) return APOLLO_OK;   // nothing has run; the status word is not initialised yet
    if (cudaMemcpy(&word, ctx->d_status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return APOLLO_ERR_CUDA;
    if (word != STATUS_OK) {
        cudaMemset(ctx->d_status, 0, 2 * sizeof(word));      // the status word and the record of the wait that gave up
        return word == STATUS_BOUNDS ? APOLLO_ERR_INTERNAL : APOLLO_ERR_TIMEOUT;
    }
    return APOLLO_OK;
}

static size_t state_elem_bytes(const apollo_ctx* ctx) { return (ctx->cfg.flags & APOLLO_FLAG_BF16_STATES) ? 2 : sizeof(float); }

// Checkpoint layout: for each matrix in list order M (r x n floats), V (r x n floats), then one
// float: the limiter's previous norm.
int apollo_state_bytes(const apollo_ctx* ctx, size_t* out_bytes)
{
    if (!ctx || !out_bytes) return APOLLO_ERR_INVALID_ARG;
    size_t total = 0;
    for (int i = 0; i < ctx->n_mat; ++i)
        total += state_elem_bytes(ctx) * 2 * (size_t)ctx->cfg.rank * (size_t)ctx->h_descs[i].n + sizeof(float);
    *out_bytes = total;
    return APOLLO_OK;
}

static int state_copy(apollo_ctx* ctx, char* d_flat, bool to_flat, cudaStream_t stream)
{
    if (((uintptr_t)d_flat % state_elem_bytes(ctx)) != 0) return APOLLO_ERR_ALIGN;
    size_t at = 0;
    for (int i = 0; i < ctx->n_mat; ++i) {
        const MatDesc& d = ctx->h_descs[i];
        // M and V are dense (r x n) in the checkpoint and have row pitch ns in the workspace
        const size_t row = state_elem_bytes(ctx) * (size_t)d.n, pitch = state_elem_bytes(ctx) * (size_t)d.ns;
        const size_t r = (size_t)ctx->cfg.rank;
        void* parts[2] = { d.M, d.V };
        for (int k = 0; k < 2; ++k) {
            if (d.state_tiled) {
                const int esz = (int)state_elem_bytes(ctx);
                launch_state_copy(parts[k], d_flat + at, (int)r, ctx->plan.tc_rank, d.n, d.ns, true, esz, esz, to_flat, stream);
                if (!cuda_ok(cudaGetLastError())) return APOLLO_ERR_CUDA;
            } else {
                const cudaError_t e = to_flat
                    ? cudaMemcpy2DAsync(d_flat + at, row, parts[k], pitch, row, r, cudaMemcpyDeviceToDevice, stream)
                    : cudaMemcpy2DAsync(parts[k], pitch, d_flat + at, row, row, r, cudaMemcpyDeviceToDevice, stream);
                if (!cuda_ok(e)) return APOLLO_ERR_CUDA;
            }
            at += row * r;
        }
        const cudaError_t e = to_flat
            ? cudaMemcpyAsync(d_flat + at, d.prev, sizeof(float), cudaMemcpyDeviceToDevice, stream)
            : cudaMemcpyAsync(d.prev, d_flat + at, sizeof(float), cudaMemcpyDeviceToDevice, stream);
        if (!cuda_ok(e)) return APOLLO_ERR_CUDA;
        at += sizeof(float);
    }
    return APOLLO_OK;
}

int apollo_state_export(apollo_ctx* ctx, void* d_out, void* cuda_stream)
{
    if (!ctx || !d_out) return APOLLO_ERR_INVALID_ARG;
    if (ctx->first && !ctx->imported) return APOLLO_ERR_INVALID_ARG;   // no step has run: nothing to export yet
    return state_copy(ctx, static_cast<char*>(d_out), true, static_cast<cudaStream_t>(cuda_stream));
}

int apollo_state_import(apollo_ctx* ctx, const void* d_in, int64_t step_count, void* cuda_stream)
{
    if (!ctx || !d_in || step_count < 0) return APOLLO_ERR_INVALID_ARG;
    // what the checkpoint does not hold starts at zero: the rows that pad the rank on the tensor path, the pitch padding
    if (cudaMemsetAsync(ctx->ws + ctx->plan.zero_begin, 0, ctx->plan.zero_end - ctx->plan.zero_begin,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return APOLLO_ERR_CUDA;
    const int rc = state_copy(ctx, const_cast<char*>(static_cast<const char*>(d_in)), false,
                              static_cast<cudaStream_t>(cuda_stream));
    if (rc != APOLLO_OK) return rc;
    ctx->t = step_count;
    ctx->imported = true;
    ctx->staged_epoch.assign((size_t)ctx->n_mat, -1);
    return APOLLO_OK;
}

int apollo_set_projection(apollo_ctx* ctx, int32_t matrix, const float* d_P)
{
    if (!ctx || matrix < 0 || matrix >= ctx->n_mat) return APOLLO_ERR_INVALID_ARG;
    if (d_P && ((uintptr_t)d_P % 4)) return APOLLO_ERR_ALIGN;
    MatDesc& d = ctx->h_descs[matrix];
    if (d_P && d.path == PATH_TENSOR && !ctx->plan.tc.staged) return APOLLO_ERR_UNSUPPORTED;
    d.ext_p = d_P;
    ctx->staged_epoch[matrix] = -1;
    d.r_scale = d_P ? 1.0f : (float)(1.0 / std::sqrt((double)ctx->cfg.rank));
    ctx->descs_dirty = true;
    return APOLLO_OK;
}

int apollo_set_timing(apollo_ctx* ctx, int32_t on)
{
    if (!ctx) return APOLLO_ERR_INVALID_ARG;
    if (on && !ctx->timing_ready) {
        for (int sl = 0; sl < APOLLO_TIMING_SLOTS; ++sl)
            for (int e = 0; e < 4; ++e)
                if (cudaEventCreate(&ctx->ev[sl][e]) != cudaSuccess) return APOLLO_ERR_CUDA;
        ctx->timing_ready = true;
    }
    ctx->timing_on = on != 0;
    return APOLLO_OK;
}

int apollo_get_timing(apollo_ctx* ctx, int32_t steps_back, float* h_ms)
{
    if (!ctx || !h_ms || !ctx->timing_ready || steps_back < 0 || steps_back >= APOLLO_TIMING_SLOTS ||
        steps_back >= ctx->t)
        return APOLLO_ERR_INVALID_ARG;
    cudaEvent_t* ev = ctx->ev[(ctx->t - 1 - steps_back) % APOLLO_TIMING_SLOTS];
    if (cudaEventSynchronize(ev[3]) != cudaSuccess) return APOLLO_ERR_CUDA;
    for (int e = 0; e < 3; ++e)
        if (cudaEventElapsedTime(h_ms + e, ev[e], ev[e + 1]) != cudaSuccess) return APOLLO_ERR_CUDA;
    if (cudaEventElapsedTime(h_ms + 3, ev[0], ev[3]) != cudaSuccess) return APOLLO_ERR_CUDA;
    return APOLLO_OK;
}

int apollo_get_path(const apollo_ctx* ctx, int32_t matrix, int32_t* out)
{
    if (!ctx || !out || matrix < 0 || matrix >= ctx->n_mat) return APOLLO_ERR_INVALID_ARG;
    *out = ctx->h_descs[matrix].path;
    return APOLLO_OK;
}

int apollo_last_launches(const apollo_ctx* ctx, int32_t* out)
{
    if (!ctx || !out) return APOLLO_ERR_INVALID_ARG;
    *out = ctx->last_launches;
    return APOLLO_OK;
}

int apollo_philox_draws(uint64_t seed, uint32_t matrix, uint32_t epoch, int32_t r, int32_t m,
                        uint32_t* d_out, void* cuda_stream)
{
    if (!d_out || r < 1 || m < 1) return APOLLO_ERR_INVALID_ARG;
    if ((uintptr_t)d_out % 16) return APOLLO_ERR_ALIGN;
    launch_philox_draws((uint32_t)(seed & 0xFFFFFFFFull), (uint32_t)(seed >> 32), matrix, epoch, r, m, d_out,
                        static_cast<cudaStream_t>(cuda_stream));
    return cudaGetLastError() == cudaSuccess ? APOLLO_OK : APOLLO_ERR_CUDA;
}

int apollo_projection(uint64_t seed, uint32_t matrix, uint32_t epoch, int32_t r, int32_t m,
                      float* d_out, void* cuda_stream)
{
    if (!d_out || r < 1 || m < 1) return APOLLO_ERR_INVALID_ARG;
    launch_projection((uint32_t)(seed & 0xFFFFFFFFull), (uint32_t)(seed >> 32), matrix, epoch, r, m, d_out,
                      static_cast<cudaStream_t>(cuda_stream));
    return cudaGetLastError() == cudaSuccess ? APOLLO_OK : APOLLO_ERR_CUDA;
}

}  // extern "C"
