// Host-callable launchers of the kernels (one grouped launch each over the parameter list).
#pragma once
#include "../../include/apollo.h"
#include "apollo_internal.h"

namespace apollo {

void launch_philox_draws(uint32_t key0, uint32_t key1, uint32_t matrix, uint32_t epoch, int r, int m,
                         uint32_t* d_out, cudaStream_t stream);
void launch_projection(uint32_t key0, uint32_t key1, uint32_t matrix, uint32_t epoch, int r, int m,
                       float* d_out, cudaStream_t stream);
void launch_project_stream(int dtype, const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                           const StepParams& sp, int sm_count, int32_t* d_status, cudaStream_t stream);
void launch_project_simt(int dtype, const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                         const StepParams& sp, int sm_count, int32_t* d_status, cudaStream_t stream);
// d_status (may be null): the context's status word.  When it is not STATUS_OK -- a bounded wait of the
// projection gave up -- finalize and update return without writing, so that a step whose projection is
// incomplete leaves the weights, the scales and the limiter's norm as they were.  Kernels built with
// -DAPOLLO_DEBUG also report a failed index check there (STATUS_BOUNDS).
void launch_finalize(const MatDesc* d_descs, int first, int count, const StepParams& sp, int32_t* d_status,
                     cudaStream_t stream);
void launch_update(int dtype, const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                   const StepParams& sp, int sm_count, int32_t* d_status, cudaStream_t stream);


// bfloat16 -> float copy (observability of bfloat16 states).
// Copies a moment between the library's layout (state_at(): row-major with pitch ns, or channel blocks of
// 128) and dense r x n rows; lib_esz / dense_esz are 2 (bfloat16) or 4 (fp32), a bfloat16 source is
// widened when the destination is fp32.  to_dense = false copies dense -> library (same element size).
// rank_layout: rows the library's layout was planned with (the padded rank on the tensor path); `rank` rows are copied.
void launch_state_copy(void* d_lib, void* d_dense, int rank, int rank_layout, int n, int ns, bool tiled, int lib_esz,
                       int dense_esz, bool to_dense, cudaStream_t stream);
// The rank the tensor path works with: `rank` rounded up to a multiple of 16 (32 above 256).
int tensor_path_padded_rank(int rank);

// Tensor-core projection (TMA + tcgen05 + TMEM).
bool tensor_path_supports(int rows, int cols, int rank, int dtype, const TcTiling& tl);
// The tiling and mode for a rank, the context's flags and the caller's tuning (may be null):
// APOLLO_OK, or APOLLO_ERR_INVALID_ARG for a tuning value out of range.
int tensor_path_configure(int rank, uint32_t flags, const apollo_tuning* tuning, TcTiling* out);
// Whether the pair kernel re-aligns this matrix's G tiles in shared memory instead of reading a padded copy.
bool tensor_path_raw_ok(int rows, int cols, const TcTiling& tl);
// Switches the tiling to the stage layout that such matrices need (fewer, larger stages).
void tensor_path_enable_raw(TcTiling* tl);
void tensor_path_tiling(int rows, int cols, int rank, const TcTiling& tl, int32_t* tiles_n, int32_t* tiles_k,
                        int32_t* slices, int32_t* g2_slices);
// Bytes one matrix's P needs in the scratch (rank x round_up(m, 64) bf16).
size_t tensor_path_stage_bytes(int rows, int cols, int rank, bool split);
// Bytes of the bfloat16 high/low copy of an fp32 gradient, and its row pitch in elements.
size_t tensor_path_split_bytes(int rows, int cols, int* pitch);
// Writes those copies for matrices [first, first + count) and the squared column norms of the gradients.
void launch_split(const MatDesc* d_descs, int first, int count, cudaStream_t stream);
// Encodes the tensor maps of the matrices on the tensor path (G at +0, the P slot at +128 of
// each 256-byte slot) into h_maps (2 x n_mat maps of 128 bytes, host).  Returns an APOLLO_* code.
int tensor_path_prepare(MatDesc* h_descs, int n_mat, int rank, const TcTiling& tl, void* h_maps);
// Copies the gradients whose row pitch is not a multiple of 16 bytes into their padded buffers.
void launch_repitch(const MatDesc* d_descs, int first, int count, cudaStream_t stream);
// Test hook: a bounded wait that is left to run out (sets STATUS_TIMEOUT in *d_status).
void launch_bounded_wait_selftest(int32_t* d_status, cudaStream_t stream);
// Fills the P slots of matrices [mat_begin, mat_end) with their standard normals (generate_p_kernel).
void launch_generate_p(const MatDesc* d_descs, int mat_begin, int mat_end, const StepParams& sp, cudaStream_t stream);
// Projection over tiles [tile_begin, tile_end) of the tensor-path prefix table.
void launch_project_tensor(const MatDesc* d_descs, const int* d_prefix, int n_mat, int tile_begin, int tile_end,
                           const StepParams& sp, const TcTiling& tl, const GenArgs& gen, TcLaunchState& state,
                           int sm_count, int32_t* d_status, cudaStream_t stream);

}  // namespace apollo
