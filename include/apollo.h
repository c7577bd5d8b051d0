/*
 * libapollo -- the APOLLO / APOLLO-Mini optimizer step on NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer argument is tagged HOST or DEVICE below.  Every function returns
 * APOLLO_OK (0) or a negative APOLLO_ERR_* code; nothing is launched when validation
 * fails; no exception crosses this boundary.  The library allocates no device memory: the
 * caller owns the weights, the gradients and one workspace buffer and keeps them alive
 * for the lifetime of the context.
 *
 * The method (Zhu et al., "APOLLO: SGD-like Memory, AdamW-level Performance",
 * Algorithm 1).  For each 2-D weight W with gradient G, viewed as m x n with m <= n
 * (m = the shorter stored side; on a tie the rows are the projected side):
 *   1. P (r x m), entries N(0, 1/r), is regenerated from a counter-based Philox4x32-10
 *      stream keyed by the seed, with counter (column quad, row, matrix index,
 *      epoch = floor(t / T)); it is regenerated in every step and not kept from one step
 *      to the next unless APOLLO_FLAG_KEEP_P asks for it (Algorithm 1, "P_t <- N_seed(0, 1/r)";
 *      Section "Generating random projection matrix").  P has the precision of the
 *      projection's operands: its standard normals are rounded to bfloat16 for bf16
 *      gradients at rank > 1; for fp32 gradients and at rank 1 they are fp32 (on the tensor
 *      cores: a bfloat16 high part plus a bfloat16 low part, 16 mantissa bits, like G).
 *   2. R = P G  (r x n)                                        (Algorithm 1, step 1).
 *   3. M <- beta1 M + (1-beta1) R,  V <- beta2 V + (1-beta2) R^2,
 *      R~ = M / (sqrt(V) + eps)                                (Algorithm 1, step 2).
 *   4. channel mode: s_j = |R~[:,j]| / |R[:,j]|                (Eq. 5);
 *      tensor mode (APOLLO-Mini): s = |R~|_F / |R|_F           (Section on APOLLO-Mini);
 *      norm-growth limiter on the scaled gradient G diag(s)    (Eq. 4): if its
 *      Frobenius norm exceeds gamma times the previous step's (limited) norm it is
 *      rescaled by c = gamma * prev / norm.
 *   5. W <- W - lr (alpha c s_j G_ij + wd W_ij)                (Algorithm 1, step 4;
 *      G is the gradient of the loss, so the update subtracts).
 */
#ifndef APOLLO_H_
#define APOLLO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define APOLLO_API __attribute__((visibility("default")))
#else
#define APOLLO_API
#endif

#define APOLLO_OK 0
#define APOLLO_ERR_INVALID_ARG (-1) /* null pointer, non-finite scalar, bad enum, bad index */
#define APOLLO_ERR_SHAPE (-2)       /* rows or cols < 1, or a side above 2^31 - 1 */
#define APOLLO_ERR_RANK (-3)        /* rank < 1, rank > min(rows, cols) or rank > APOLLO_MAX_RANK */
#define APOLLO_ERR_ALIGN (-4)       /* a device pointer is not 16-byte aligned */
#define APOLLO_ERR_WORKSPACE (-5)   /* workspace smaller than apollo_workspace_bytes() */
#define APOLLO_ERR_CUDA (-6)        /* a CUDA runtime or driver call failed */
#define APOLLO_ERR_TIMEOUT (-7)     /* a bounded device-side wait expired (reported by apollo_status) */
#define APOLLO_ERR_UNSUPPORTED (-8) /* the device is not an sm_100 part */
#define APOLLO_ERR_TOO_LARGE (-9)   /* the matrix does not fit the built-in scratch of apollo_mini_step_static */
#define APOLLO_ERR_INTERNAL (-10)   /* debug build of the library (-DAPOLLO_DEBUG) only: an index check inside a kernel
                                       failed; the access was skipped (reported by apollo_status) */

#define APOLLO_MAX_RANK 512

#define APOLLO_SCALE_CHANNEL 0 /* APOLLO: one scale per channel (Eq. 5) */
#define APOLLO_SCALE_TENSOR 1  /* APOLLO-Mini: one scale per tensor (use with rank 1) */

#define APOLLO_DT_F32 0  /* W and G are float */
#define APOLLO_DT_BF16 1 /* W and G are bfloat16; W is stored with round-to-nearest-even */

/* apollo_config.flags */
#define APOLLO_FLAG_NO_TENSOR_CORES 1u /* run the projection on the CUDA cores (test and comparison aid) */
#define APOLLO_FLAG_BF16_STATES 2u     /* keep M and V in bfloat16 (two bytes per entry, as the paper's state-size
                                          figures assume); R~ is formed from the unrounded update */
#define APOLLO_FLAG_KEEP_P 4u          /* tensor-core path: keep every matrix's projection (r x m bfloat16) in the
                                          workspace for the T steps of its epoch instead of regenerating it from the
                                          seed in every step.  Off by default: the method keeps only the seed
                                          (Algorithm 1; the paper's state-size table counts 2nr + 2 per matrix) */

typedef struct apollo_ctx apollo_ctx; /* opaque HOST object */

typedef struct {
    int64_t rows, cols; /* stored shape, row-major, contiguous (pitch = cols elements) */
} apollo_shape;

typedef struct {
    int32_t rank;            /* r */
    int32_t mode;            /* APOLLO_SCALE_* */
    int32_t dtype;           /* APOLLO_DT_* of W and G; M, V, s and all reductions are fp32 */
    int32_t T;               /* projection refresh period in steps, >= 1 (paper default 200) */
    uint64_t seed;           /* Philox key */
    float alpha;             /* gradient scale factor (1 for APOLLO, sqrt(128) for Mini) */
    float gamma;             /* limiter threshold (paper default 1.01); <= 0 disables the limiter */
    float beta1, beta2, eps; /* 0.9, 0.999, 1e-8 */
    int32_t bias_correction; /* 0: moment equations as printed; 1: divide by 1-beta^t as Adam does */
    uint32_t flags;          /* APOLLO_FLAG_* */
} apollo_config;

/*
 * Tuning of the tensor-core projection, fixed when a context is created (and when its workspace is
 * sized: pass the same values to both calls).  A zeroed struct, or a NULL pointer, selects the
 * defaults.  None of the fields changes the results beyond the order of floating-point sums.
 */
#define APOLLO_TC_KERNEL_PAIR 0 /* CTA pairs share every MMA (tcgen05 cta_group::2); default */
#define APOLLO_TC_KERNEL_RING 1 /* one CTA per tile, single shared-memory ring */
#define APOLLO_P_SCRATCH 0      /* P goes through a scratch in the workspace that L2 keeps (default) */
#define APOLLO_P_SHARED 1       /* every CTA generates the P tiles it needs straight into shared memory (ring kernel) */
typedef struct {
    int32_t kernel;        /* APOLLO_TC_KERNEL_* */
    int32_t p_source;      /* APOLLO_P_* */
    int32_t p_generator;   /* with APOLLO_P_SCRATCH and without APOLLO_FLAG_KEEP_P: 0 = default: a list whose projections
                              all fit the scratch is refilled by one launch of the generator kernel per step, a
                              larger one by spare warps of the pair kernel, a few matrices ahead of their use,
                              through a ring of slots; 1 = always the generator kernel, group by group between
                              projection launches; 2 = always the spare warps */
    int32_t scratch_mb;    /* most the P scratch may take, in MB; 0 = default (128).  A list whose projections all
                              fit is regenerated into it by one launch of the generator kernel per step; a larger
                              list goes through a ring of at most 32 MB of it (see p_generator) */
    int32_t r_slice;       /* rows of R per tile: a multiple of 16, <= 256, that divides the rank rounded up to a
                              multiple of 16 (32 above 256); 0 = default */
    int32_t nblk;          /* ring kernel: 128-channel blocks per tile (1, 2 or 4; nblk * r_slice <= 512); 0 = default */
    int32_t epi_prefetch;  /* pair kernel: how many 16-row chunks ahead of its loads an epilogue warp asks L2 for
                              the moments, as distance + 1 (1 = no prefetch ... 9 = eight chunks); 0 = default (one chunk) */
    int32_t realign;       /* gradients whose rows start on no 16-byte boundary (cols % 8 != 0), which no tensor map
                              can describe: 0 (default) and 2 = all of them are first copied to a padded pitch (rows x
                              round_up(cols, 8) bf16 per matrix, see repitch_mb); 1 = wide ones with rows % 8 == 0
                              are instead fetched as they lie and re-aligned in shared memory by the pair kernel: no
                              extra memory (LLaMA-1B list: -1.07 GB of workspace, +5 % per step) */
    int32_t repitch_mb;    /* workspace for those padded copies in MB; 0 = no limit: every such matrix has its own copy
                              and the list is projected by one launch (default, fastest).  With a limit the matrices
                              share the buffer group by group in list order: each group is copied, then projected, by
                              launches of its own (LLaMA-1B list, 256 MB: -0.83 GB of workspace, +4 % per step) */
} apollo_tuning;

/*
 * Bytes of DEVICE workspace a context over `shapes[0..n_matrices)` needs: moments, scales,
 * partial sums, descriptor tables, tensor maps, and for the tensor-core path a scratch for the
 * random projections.  By default that scratch holds a few matrices' projections (32 MB; all of
 * them when they fit in 128 MB) and is refilled from the seed in every step (Algorithm 1 "P_t <- N_seed(0, 1/r)": only the seed is
 * kept).  With APOLLO_FLAG_KEEP_P every matrix has its own r x m slot, filled in the step that
 * opens an epoch (every T steps, Algorithm 1 "if t mod T = 0") and read again by the following
 * steps of the epoch; the steps of such a context must reach the GPU in order, whatever streams
 * they use.  shapes, cfg, tuning (may be NULL), out: HOST.
 */
APOLLO_API int apollo_workspace_bytes(const apollo_shape* shapes, int32_t n_matrices, const apollo_config* cfg,
                           size_t* out_bytes);
APOLLO_API int apollo_workspace_bytes_tuned(const apollo_shape* shapes, int32_t n_matrices, const apollo_config* cfg,
                                            const apollo_tuning* tuning, size_t* out_bytes);

/*
 * Create a context (Algorithm 1, "Initialize: t <- 0").  d_workspace: DEVICE, 256-byte
 * aligned, workspace_bytes >= apollo_workspace_bytes(); owned by the caller, used
 * exclusively by this context until apollo_destroy.  Launches nothing and touches no
 * stream: the moments are zeroed (Appendix: "zero initialization") by the first
 * apollo_step on that step's stream.  The matrix index in the list is the `matrix index`
 * word of the Philox counter.  Must be called with the target device current.  The library
 * reads no environment variable.  apollo_create is apollo_create_tuned with tuning = NULL;
 * a tuning value out of range is APOLLO_ERR_INVALID_ARG.
 */
APOLLO_API int apollo_create(apollo_ctx** out_ctx, const apollo_shape* shapes, int32_t n_matrices,
                  const apollo_config* cfg, void* d_workspace, size_t workspace_bytes);
APOLLO_API int apollo_create_tuned(apollo_ctx** out_ctx, const apollo_shape* shapes, int32_t n_matrices,
                                   const apollo_config* cfg, const apollo_tuning* tuning, void* d_workspace,
                                   size_t workspace_bytes);

/*
 * One optimizer step over the whole parameter list (Algorithm 1, body of the loop).
 * d_W, d_G: HOST arrays of n_matrices DEVICE pointers (16-byte aligned, dtype of the
 * config, row-major rows x cols).  W is updated in place; G is read only.  lr and wd are
 * the step size eta and the weight decay lambda.  Asynchronous on `cuda_stream`
 * (a cudaStream_t; NULL = the legacy default stream); no host synchronisation; advances
 * the step counter t.  Not thread-safe per context.
 */
APOLLO_API int apollo_step(apollo_ctx* ctx, void* const* d_W, const void* const* d_G, float lr, float wd,
                void* cuda_stream);

/*
 * The same step for matrices [first, first + count) only, at the current step counter
 * (d_W, d_G: HOST arrays of `count` DEVICE pointers).  This is what a layer-wise update
 * strategy needs (the paper's Figure 1 caption and its paragraph on training under 12 GB:
 * run the optimizer for a layer as soon as its gradient exists and free the gradient): call it once per layer during the backward
 * pass, in any order, each matrix exactly once per step, and pass close_step != 0 on the
 * last call of the step so that t advances.  apollo_step is apollo_step_range over the
 * whole list with close_step = 1.
 */
APOLLO_API int apollo_step_range(apollo_ctx* ctx, int32_t first, int32_t count, void* const* d_W,
                                 const void* const* d_G, float lr, float wd, int32_t close_step, void* cuda_stream);

APOLLO_API int apollo_destroy(apollo_ctx* ctx);

/* Number of steps taken so far (t of Algorithm 1).  out: HOST. */
APOLLO_API int apollo_step_count(const apollo_ctx* ctx, int64_t* out);

/*
 * Observability (used by the tests).  All copies are asynchronous on `cuda_stream`.
 * apollo_get_scales:  d_out DEVICE, n floats: s_j of the last step (Eq. 5), n = max(rows, cols).
 * apollo_get_limiter: d_out DEVICE, 4 floats: {norm after limiting (Eq. 4), factor c,
 *                     norm before limiting, tensor-wise scale (tensor mode, else 0)}.
 * apollo_get_state:   d_M, d_V DEVICE, r x n floats each, row-major (channel index contiguous);
 *                     bfloat16 states are widened to float.
 */
APOLLO_API int apollo_get_scales(apollo_ctx* ctx, int32_t matrix, float* d_out, void* cuda_stream);
APOLLO_API int apollo_get_limiter(apollo_ctx* ctx, int32_t matrix, float* d_out, void* cuda_stream);
APOLLO_API int apollo_get_state(apollo_ctx* ctx, int32_t matrix, float* d_M, float* d_V, void* cuda_stream);

/*
 * Optional capture of the fp32 update dW = -lr (alpha c s_j G_ij + wd W_ij) before it is
 * added to W and rounded (the quantity the parity bound is stated on).  d_dW: HOST array
 * of n_matrices DEVICE pointers (rows x cols floats each; a null entry leaves that matrix
 * uncaptured), or NULL to switch capture off.
 */
APOLLO_API int apollo_set_delta_out(apollo_ctx* ctx, float* const* d_dW);

/*
 * Synchronises `cuda_stream` and returns the device status word, clearing it: APOLLO_OK, or
 * APOLLO_ERR_TIMEOUT if a bounded wait inside a projection kernel expired since the last call
 * (APOLLO_ERR_INTERNAL: see above).  While the word is set, the finalize and update passes of
 * every step write nothing: the step whose projection gave up, and the steps issued after it
 * until this call, leave the weights, the scales and the limiter's norm as they were.  The
 * moments of that step are partly updated; resume from a checkpoint (apollo_state_import) to
 * continue exactly.
 */
APOLLO_API int apollo_status(apollo_ctx* ctx, void* cuda_stream);

/*
 * The generator by itself (Algorithm 1, "P_t <- N_seed(0, 1/r)"), for tests.
 * apollo_philox_draws:  d_out DEVICE, r x ceil(m/4) x 4 uint32: the raw Philox4x32-10
 *                       words for counter (q, k, matrix, epoch), key = seed.
 * apollo_projection:    d_out DEVICE, r x m floats: the standard normals Z behind P
 *                       (P = Z / sqrt(r)) in fp32, before any rounding to bfloat16.
 */
APOLLO_API int apollo_philox_draws(uint64_t seed, uint32_t matrix, uint32_t epoch, int32_t r, int32_t m,
                        uint32_t* d_out, void* cuda_stream);
APOLLO_API int apollo_projection(uint64_t seed, uint32_t matrix, uint32_t epoch, int32_t r, int32_t m,
                      float* d_out, void* cuda_stream);

/* Which projection kernel a matrix was assigned: 0 streaming (rank 1), 1 CUDA cores, 2 tensor cores. */
APOLLO_API int apollo_get_path(const apollo_ctx* ctx, int32_t matrix, int32_t* out);

/*
 * A projection supplied by the caller instead of the seeded Gaussian one: the paper's
 * "APOLLO w. SVD" variant takes P from a decomposition of the gradient and notes that it
 * works as well at a much higher cost; the decomposition is the caller's business, this call
 * only swaps the operand.  d_P: DEVICE, r x m floats, row-major (m = min(rows, cols)), used
 * as is (R = P G, no 1/sqrt(r) factor) in every later step until replaced; NULL returns
 * the matrix to the generator.  For bf16 gradients at rank > 1, P is rounded to bfloat16 as
 * the generated one is.  The buffer stays owned by the caller and must stay alive.  Not
 * available with APOLLO_P_SHARED (APOLLO_ERR_UNSUPPORTED).
 */
APOLLO_API int apollo_set_projection(apollo_ctx* ctx, int32_t matrix, const float* d_P);

/*
 * Checkpoint and resume.  The optimizer state of Algorithm 1 is, per matrix, the moments M^R
 * and V^R, the limiter's previous norm, the seed and the step counter t (the paper's table of
 * state sizes: "2nr + 2"); P is not part of it because it is regenerated from (seed, matrix
 * index, floor(t / T)).  apollo_state_bytes gives the size of the flat DEVICE buffer:
 * per matrix in list order M (r x n entries), V (r x n entries), one float (previous norm);
 * entries are floats, or bfloat16 with APOLLO_FLAG_BF16_STATES; the buffer is aligned to the entry
 * size (APOLLO_ERR_ALIGN otherwise) and holds dense row-major matrices whatever layout the
 * library keeps them in, so it can be read by a context that uses another projection kernel.
 * apollo_state_export copies the state out (after at least one step or an import);
 * apollo_state_import copies it in and sets the step counter; the context must have been
 * created with the same shapes and configuration (the seed and t are the caller's to keep:
 * read t with apollo_step_count).  Both are asynchronous on `cuda_stream`.  A resumed run
 * continues bit for bit like the uninterrupted one.
 */
APOLLO_API int apollo_state_bytes(const apollo_ctx* ctx, size_t* out_bytes);
APOLLO_API int apollo_state_export(apollo_ctx* ctx, void* d_out, void* cuda_stream);
APOLLO_API int apollo_state_import(apollo_ctx* ctx, const void* d_in, int64_t step_count, void* cuda_stream);

/*
 * Per-phase device timing.  apollo_set_timing(ctx, 1) makes every later apollo_step record
 * CUDA events on its stream around the three phases (projection, finalize, update); the
 * last APOLLO_TIMING_SLOTS steps are kept.  apollo_get_timing waits for the chosen step
 * (steps_back = 0 is the last one) and writes {projection, finalize, update, whole step}
 * in milliseconds to h_ms (HOST, 4 floats).
 */
#define APOLLO_TIMING_SLOTS 64
APOLLO_API int apollo_set_timing(apollo_ctx* ctx, int32_t on);
APOLLO_API int apollo_get_timing(apollo_ctx* ctx, int32_t steps_back, float* h_ms);

/*
 * AdamW for the parameters the method does not project (embeddings, norms, output head;
 * the paper states APOLLO for 2-D weight matrices and keeps the base optimizer elsewhere).
 * Eq. 1 with decoupled weight decay:  m <- b1 m + (1-b1) g,  v <- b2 v + (1-b2) g^2,
 *   p <- p - lr ((m / c1) / (sqrt(v / c2) + eps) + wd p),  c_i = 1 - b_i^(t+1) with
 * bias_correction = 1 (the usual AdamW), c_i = 1 with 0 (Eq. 1 as printed).
 * d_P, d_G, d_M, d_V: HOST arrays of n_tensors DEVICE pointers (16-byte aligned); P and G
 * have `dtype` (APOLLO_DT_*), M and V are fp32 of the same length, owned and zero-initialised
 * by the caller; numel: HOST.  t = steps already taken.  d_dP: optional HOST array of DEVICE
 * fp32 buffers that receive the update before it is added and rounded (entries or the array
 * may be NULL).  Stateless, needs no workspace, asynchronous on `cuda_stream`.
 */
APOLLO_API int apollo_adamw_step(void* const* d_P, const void* const* d_G, float* const* d_M, float* const* d_V,
                                 const int64_t* numel, int32_t n_tensors, int32_t dtype, float lr, float beta1,
                                 float beta2, float eps, float wd, int64_t t, int32_t bias_correction,
                                 float* const* d_dP, void* cuda_stream);

/*
 * A rank-1 step for one matrix that allocates nothing and needs no workspace.  (The
 * paper has no counterpart to this entry point; it computes exactly what apollo_step
 * computes for a one-matrix list with rank 1.)
 *
 * Who it is for: code that is not allowed to obtain device memory at the point where it
 * has to run the optimizer -- a plug-in running inside another runtime's memory plan, a
 * real-time loop that must not hit the synchronisation a device allocation implies, a
 * process whose memory pool is already handed out in full.  Such callers cannot provide
 * apollo_create's workspace either.  Here the caller passes only the method's own inputs
 * and outputs; the temporaries (descriptor, tile tables, partial sums of the projection,
 * the n scales, limiter scalars) live in a fixed array of APOLLO_STATIC_SCRATCH_BYTES that
 * is part of the library image: every GPU that loads the library holds it until exit.
 *
 *   d_W, d_G      DEVICE, rows x cols of cfg->dtype, 16-byte aligned; W updated in place.
 *   d_M, d_V      DEVICE, n = max(rows, cols) floats each, 16-byte aligned: the rank-1
 *                 moments, owned and kept by the caller between steps (zero them before
 *                 the first step).
 *   d_prev_norm   DEVICE, one float: the limiter's previous norm (Eq. 4), in and out;
 *                 zero before the first step.
 *   cfg           HOST; cfg->rank must be 1 (APOLLO_ERR_RANK otherwise); mode, dtype, T,
 *                 seed, alpha, gamma, betas, eps, bias_correction as for apollo_create.
 *                 The moments are floats here: APOLLO_FLAG_BF16_STATES is rejected
 *                 (APOLLO_ERR_INVALID_ARG); the other flags have no meaning at rank 1.
 *   matrix, t     the matrix index word of the Philox counter and the number of steps
 *                 already taken (the caller keeps t; epoch = t / T).
 * Limits and rules: the temporaries are 1 KiB of tables, the n scales (4 n bytes) and the
 * partial sums of the projection (8 n ceil(rows/512) bytes for a wide matrix, 8 n for a tall
 * one), the two arrays each rounded up to a multiple of 256 bytes.  A matrix for which that
 * sum exceeds the array is rejected with APOLLO_ERR_TOO_LARGE and nothing is launched.  No cudaMalloc, cudaFree or other
 * allocating call is made.  The first call on each device looks up the array's device
 * address (with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps whatever the previous call
 * left; each call rewrites every entry it later reads, so no clearing is needed between
 * calls, but two calls that overlap on the GPU (different streams, no ordering between
 * them) race on it and give wrong results: order them.  Asynchronous on `cuda_stream`.
 */
#define APOLLO_STATIC_SCRATCH_BYTES (8u << 20)
APOLLO_API int apollo_mini_step_static(void* d_W, const void* d_G, int64_t rows, int64_t cols,
                                       float* d_M, float* d_V, float* d_prev_norm,
                                       const apollo_config* cfg, uint32_t matrix, int64_t t,
                                       float lr, float wd, void* cuda_stream);

/* Self-test of the error path (the paper has no counterpart).  Every wait inside the tensor-core
 * kernel is bounded: after 2^20 polls it gives up, sets the context's device status word and the
 * kernel winds down instead of hanging.  This call launches, on the stream, a one-block kernel whose
 * only wait can never be satisfied, so that the mechanism can be checked on a healthy GPU: the next
 * apollo_status(ctx) returns APOLLO_ERR_TIMEOUT (and clears the word), and the context works on as
 * before.  It moves no data and touches no state of the optimizer.  ctx must have run a step (the
 * status word is set up by the first step), else APOLLO_ERR_INVALID_ARG.  The wait takes of the
 * order of a second of GPU time before it gives up. */
APOLLO_API int apollo_selftest_bounded_wait(apollo_ctx* ctx, void* cuda_stream);

/* Kernel launches issued by the last apollo_step (HOST counter). */
APOLLO_API int apollo_last_launches(const apollo_ctx* ctx, int32_t* out);

APOLLO_API const char* apollo_strerror(int code);

/* Text of the last CUDA error this library saw on the calling thread ("no error" if none);
 * the detail behind an APOLLO_ERR_CUDA return. */
APOLLO_API const char* apollo_cuda_error_string(void);

#ifdef __cplusplus
}
#endif
#endif /* APOLLO_H_ */
