// Structures shared by the host side of libapollo and its kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace apollo {

// Which projection kernel serves a matrix.
enum Path : int32_t {
    PATH_STREAM = 0,  // rank 1: streaming matrix-vector pass, moments updated by the finalize kernel
    PATH_SIMT = 1,    // any rank, any dtype, any pitch: CUDA-core tiles
    PATH_TENSOR = 2,  // bf16, rank >= 16 (worked on rounded up to a multiple of 16): TMA + tcgen05 + TMEM
};

constexpr int STREAM_ROWS = 512;     // rows of a wide matrix one streaming tile covers
constexpr int STREAM_COLS = 256;     // columns of a wide matrix one streaming tile covers
constexpr int STREAM_TALL_ROWS = 64; // rows of a tall matrix one streaming tile covers
constexpr int SIMT_BN = 64;          // channels per CUDA-core tile
constexpr int SIMT_BR = 64;          // rows of R per CUDA-core tile
constexpr int SIMT_BK = 32;          // contraction chunk of the CUDA-core tile
constexpr int UPDATE_TILE = 16384;   // elements one tile of the update pass covers
// Matrices whose rows are whole 8-element vectors are updated in 2-D tiles: the columns are cut into
// equal chunks of at most UPDATE_COLS, a thread owns eight columns of a chunk (so it keeps its column
// scales in registers and no index arithmetic is left per vector), and when a chunk needs fewer than
// all the threads, several groups of UPDATE_ROWS rows are worked on side by side.  The other matrices
// go through flat tiles of UPDATE_TILE elements, or through the same 2-D tiles over super-rows (below).
constexpr int UPDATE_ROWS = 16;
constexpr int UPDATE_COLS = 2048;
constexpr int UPDATE_BLOCK = 256;      // threads of an update block
struct UpdateTiling {
    int chunks;       // column chunks
    int width;        // columns of a chunk (multiple of 8; the last chunk may be narrower)
    int groups;       // row groups side by side in one tile
};
// Among the smallest chunk counts, the one that keeps most threads busy.
inline UpdateTiling update_tiling(int cols)
{
    UpdateTiling best{1, 8, 1};
    int best_busy = -1;
    const int cmin = (cols + UPDATE_COLS - 1) / UPDATE_COLS;
    for (int c = cmin; c < cmin + 4; ++c) {
        const int width = ((cols + c - 1) / c + 7) & ~7;
        const int tpr = width / 8, groups = UPDATE_BLOCK / tpr, busy = tpr * groups;
        if (busy > best_busy) { best_busy = busy; best = UpdateTiling{c, width, groups}; }
    }
    return best;
}
// A wide matrix whose rows are not whole vectors but whose row count is a multiple of 8 is tiled the
// same way over "super-rows" of 8 stored rows: 8 * cols elements are whole vectors, every super-row
// starts on a 16-byte boundary, and element c of a super-row belongs to column c mod cols in all of them.
inline bool update_super_rows(long long rows, long long cols, bool tall)
{
    return cols % 8 != 0 && !tall && rows % 8 == 0 && cols <= (1ll << 27);
}
inline long long update_tile_count(long long rows, long long cols, bool tall)
{
    if (update_super_rows(rows, cols, tall)) { rows /= 8; cols *= 8; }
    if (cols % 8 != 0) return (rows * cols + UPDATE_TILE - 1) / UPDATE_TILE;
    const UpdateTiling t = update_tiling((int)cols);
    const long long tile_rows = (long long)UPDATE_ROWS * t.groups;
    return (rows + tile_rows - 1) / tile_rows * t.chunks;
}

// Layout of M and V (r x n).  CUDA-core paths: row-major with the row pitch rounded up to 64 elements, so
// that every row starts a 256-byte line.  Tensor path: channel blocks of 128, each block r x 128
// row-major (block b holds channels 128 b ..): the 128 channels x r_slice rows that one CTA reads and
// writes per tile are one contiguous piece of memory instead of r_slice pieces of 512 bytes n apart.
__host__ __device__ inline int state_pitch(int n, int rank) { return rank > 1 ? (n + 63) / 64 * 64 : n; }
__host__ __device__ inline long long state_elements(int n, int rank, bool tiled)
{
    return (long long)rank * (tiled ? (n + 127) / 128 * 128 : state_pitch(n, rank));
}
__host__ __device__ inline int64_t state_at(bool tiled, int64_t ns, int rank, int k, int j)
{
    return tiled ? ((int64_t)(j >> 7) * rank + k) * 128 + (j & 127) : (int64_t)k * ns + j;
}

// Per-matrix record in device memory.  Pointers into the workspace are fixed at create
// time; W, G and dW are refreshed whenever the caller passes different addresses.
struct MatDesc {
    void* W;
    const void* G;
    float* dW;        // optional fp32 capture of the update, or nullptr
    float* M;         // r x n, element (k, j) at state_at(); fp32, or bfloat16 behind the same pointer when StepParams::state_bf16
    float* V;         // r x n
    float* s;         // n scales of the last step
    float* part;      // projection partial sums, layout depends on the path (see kernels)
    float* g2;        // squared column norms of G: g2_slices x n
    float* scal;      // {norm after limiting, c, norm before limiting, tensor-wise s}
    float* prev;      // previous limited norm (one float)
    const void* tmap; // 128-byte TMA tensor map of G in device memory (tensor path only)
    const void* tmap_p; // tensor map of this matrix's slot of the P scratch
    void* pstage;     // this matrix's slot of the P scratch: rank_pad x p_width bf16 standard normals
    const float* ext_p; // caller-supplied projection (r x m fp32, row-major) used instead of the generator, or nullptr
    void* gpad;       // copy of G with a 16-byte row pitch when cols % 8 != 0 (tensor path), else nullptr
    int32_t rows, cols;
    int32_t m, n;     // m = min(rows, cols) = projected side; n = max = number of channels
    int32_t ns;       // row pitch of M and V in elements (state_pitch) when they are row-major
    int32_t state_tiled; // 1: M and V are stored in channel blocks of 128 (tensor path), see state_at()
    int32_t tall;     // 1 if rows > cols: channels are the stored rows
    int32_t path;
    int32_t slices;   // number of partial slices in `part`
    int32_t g2_slices;
    int32_t matrix_id;
    int32_t tiles_n;  // projection tiles along the channels
    int32_t tiles_k;  // projection tiles along the other tiled axis (rows of G, or rows of R)
    int32_t m_pad;    // m rounded up to 64: row length of P in its slot (twice that for a split matrix)
    int32_t g_pitch;  // row pitch (elements) of the array the tensor path reads: cols, or cols rounded up to 8
    int32_t split;    // 1: fp32 gradient on the tensor path: `gpad` holds its bfloat16 high and low parts ([hi; lo] along the
                      //    projected side, m_pad apart), the P slot holds [P_hi | P_lo], and a tile's contraction runs over
                      //    three segments (P_hi G_hi, P_lo G_hi, P_hi G_lo)
    int32_t p_width;  // elements per row of the P slot: m_pad, or 2 m_pad for a split matrix
    int32_t raw;      // 1: wide matrix with cols % 8 != 0 and rows % 8 == 0 on the pair kernel: its G tiles are fetched
                      //    as they lie in memory and re-aligned in shared memory (no padded copy)
    int32_t upd_chunks, upd_width, upd_groups;   // 2-D tiling of the update pass (update_tiling(cols)); 0 chunks: flat tiles
    int32_t upd_super;   // 1: the 2-D tiles run over super-rows of 8 stored rows (update_super_rows)
    float r_scale;    // factor applied to the contraction: 1/sqrt(r) for generated standard normals, 1 for a supplied P
};

struct StepParams {
    uint32_t key0, key1;   // Philox key = seed
    uint32_t epoch;        // floor(t / T)
    int32_t rank, mode;
    int32_t rank_pad;         // tensor path: rank rounded up to the MMA's granularity (16; 32 above 256); the rows of P
                              // from `rank` on are zero, and M and V are laid out with rank_pad rows
    float inv_sqrt_r;
    float lr, wd, alpha, gamma;
    float beta1, beta2, eps;
    float inv_bc1, inv_bc2;   // 1/(1-beta^t) with bias correction, else 1
    int32_t state_bf16;       // 1: M and V are stored as bfloat16 (APOLLO_FLAG_BF16_STATES)
    uint32_t round_key[20];   // Philox key schedule: {key0 + i W0, key1 + i W1}, i = 0..9
};

inline void fill_round_keys(StepParams& sp)
{
    for (int i = 0; i < 10; ++i) {
        sp.round_key[2 * i] = sp.key0 + (uint32_t)i * 0x9E3779B9u;
        sp.round_key[2 * i + 1] = sp.key1 + (uint32_t)i * 0xBB67AE85u;
    }
}

// Tiling and mode of the tensor-core projection: one choice per context, made when it is created.
struct TcTiling {
    int32_t r_slice;   // rows of R per tile = N of the MMA (multiple of 16, <= 256)
    int32_t nblk;      // 128-channel blocks per tile (1, 2 or 4); nblk * r_slice <= 512 TMEM columns
    int32_t stages;    // shared-memory pipeline depth
    int32_t smem_bytes;
    int32_t staged;    // 0: P generated in shared memory; 1: P loaded from the scratch in the workspace
    int32_t pair;      // 1: the pair kernel (CTA pairs, cta_group::2); staged only
    int32_t epi_prefetch; // pair kernel: the epilogue warps ask L2 for the moments this many chunks ahead of their loads
    int32_t keep;      // 1: every matrix owns a slot of the scratch, filled once per epoch (APOLLO_FLAG_KEEP_P)
    int32_t gen;       // != 0: spare warps of the pair kernel generate P into a ring of `slots` slots, ahead of its use
    int32_t slots;     // gen: slots of the ring (matrix with tensor ordinal q uses slot q % slots)
    int32_t split;     // 1: the gradients are fp32 and go through the bfloat16 high/low split (MatDesc::split)
    int32_t raw_allowed; // tuning: matrices that qualify are re-aligned in shared memory rather than copied to a padded pitch
    int32_t raw;       // 1: the list has matrices whose G tiles are re-aligned in shared memory (MatDesc::raw): the
                       //    G part of a stage is RAW_G_BYTES and the norm warps arrive on the stage's `full` barrier
    int64_t repitch_bytes; // byte budget of the padded copies of gradients with an unaligned row pitch (shared group by group)
    int64_t scratch_bytes; // byte budget of the scratch when it is neither kept nor a ring (groups of matrices share it)
};

constexpr int RAW_BOX_W = 136;                       // elements per fetched row piece: 128 channels + up to 7 of misalignment, whole 16-byte units
constexpr int RAW_G_BYTES = 64 * RAW_BOX_W * 2;      // 64 rows of a k-block as fetched: 17408 bytes (17 KiB)

// What the generator warps of the pair kernel and the consumers of their output share (TcTiling::gen).
// The counters are zeroed before every launch.
constexpr int GEN_CHUNKS = 64;     // pieces a matrix's P is generated in; one ticket each
struct GenArgs {
    const int32_t* mats;   // tensor ordinal -> matrix index
    int32_t q_begin, q_end;   // ordinals of the launch
    uint32_t* ticket;      // next piece to generate: (ordinal - q_begin) * GEN_CHUNKS + chunk
    uint32_t* gen_done;    // per matrix: pieces written
    uint32_t* use_done;    // per matrix: tiles whose MMAs have read their last P tile
};

// Per-context launch state of the tensor path (function attributes are per device; set once per context).
struct TcLaunchState {
    bool attr_set;
    int max_pairs;
};

// Device status word values.
constexpr int32_t STATUS_OK = 0;
constexpr int32_t STATUS_TIMEOUT = 1;
constexpr int32_t STATUS_BOUNDS = 2;    // debug build only: an index check inside a kernel failed (the access was skipped)

}  // namespace apollo
