/*
 * fira.h -- C ABI of the Fira optimizer update (arXiv 2410.01623) for one NVIDIA
 * B200 (sm_100a).
 *
 * What the library computes.  For every registered weight matrix W (m x n, row
 * major) and its gradient G, one call of fira_step() performs one pass of the
 * loop body of the paper's Algorithm 1 ("Fira with Adam", Appendix A.1):
 *
 *   R = P^T G,  S = (I - P P^T) G                    (Section 4.1, "Challenge analysis")
 *   M <- b1 M + (1-b1) R,  V <- b2 V + (1-b2) R^2
 *   N = sqrt(1-b2^s)/(1-b1^s) * M / (sqrt(V) + eps)   (Eq. 2-4 on R; s = steps taken incl. this one)
 *   k_i = ||N[:,i]|| / (||R[:,i]|| + eps),  S[:,i] <- k_i S[:,i]      (Eq. 11, Algorithm 1 form)
 *   S <- S * gamma / max(||S|| / (||S_prev|| + eps), gamma)            (Eq. 12, Algorithm 1 form)
 *   W <- W - lr * alpha * (P N + S)                                     (Algorithm 1, last two lines)
 *
 * Orientation.  For m <= n the projection is a left one, P is m x r and the
 * factors k are per column of G (n of them).  For m > n the footnote of Section
 * 3.3 applies: a right projection Q (n x r), R = G Q (m x r); the whole algorithm
 * is applied to the transposed problem, so the factors are per row of G (m of
 * them).  Below, d = min(m,n) is the projected extent and l = max(m,n) the other
 * one; "the projection" is the d x r matrix P or Q.
 *
 * Conventions fixed where the paper leaves a choice: the bias-correction exponent
 * is s = t + 1; the remembered norm ||S_prev|| is the norm after limiting; a
 * matrix's first step is not limited; gamma = +inf disables the limiter; a
 * projection switch keeps M, V, ||S_prev|| and t; alpha multiplies both terms
 * unless FIRA_FLAG_ALPHA_LOWRANK_ONLY is set; no weight decay.
 *
 * Memory and ownership.  Every pointer whose name ends in _dev is a device pointer
 * on the context's GPU; every other pointer is a host pointer.  The caller owns W,
 * G, the state buffer and the scratch buffer and keeps them alive for the lifetime
 * of the context; the library allocates no device memory.  The state buffer holds,
 * per matrix, the projection (d x r, row major, in the matrix's dtype), M and V
 * (each l x r, row major, float: row i belongs to column i of G when m <= n and to
 * row i of G when m > n, i.e. the transpose of the paper's r x n layout in the
 * first case), ||S_prev|| (float) and t (int64): the d r + 2 l r + 1 numbers of the
 * paper's comparison table plus the step count.  The scratch buffer holds
 * intermediates and is overwritten by every call.
 *
 * Streams and errors.  All device work is enqueued on the stream given to
 * fira_init() and calls return without waiting for it unless stated otherwise.
 * Host-side argument errors are returned at once and leave the state untouched.
 * Device-side conditions (a bounded wait that ran out, a non-finite norm) are
 * recorded in a status word that fira_poll() reads.  No entry point throws, aborts
 * or traps.  A context is not thread safe.
 */
#ifndef FIRA_H_
#define FIRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define FIRA_API __attribute__((visibility("default")))
#else
#define FIRA_API
#endif

typedef enum {
  FIRA_OK = 0,
  FIRA_ERR_INVALID_ARG = 1,
  FIRA_ERR_WORKSPACE_TOO_SMALL = 2,
  FIRA_ERR_UNSUPPORTED = 3,
  FIRA_ERR_CUDA = 4,
  FIRA_ERR_DEVICE_TIMEOUT = 5,
  FIRA_ERR_NONFINITE = 6
} fira_status;

typedef enum { FIRA_F32 = 0, FIRA_BF16 = 1 } fira_dtype;

/* fira_hparams.flags */
#define FIRA_FLAG_ALPHA_LOWRANK_ONLY 1u /* G~ = alpha P N + S instead of alpha (P N + S) */
#define FIRA_FLAG_AUTO_REFRESH 2u       /* fira_step() refreshes a matrix's projection when t mod T == 0 */
#define FIRA_FLAG_FORCE_SIMT 4u         /* bf16 matrices also use the fp32 CUDA-core kernels */
/* Ablation variants of Section 5.4 ("Ablation Study"); epilogue switches of the same kernels.  The
 * first two exclude each other. */
#define FIRA_FLAG_MATRIX_SCALING 8u     /* Fira-matrix: one factor ||N||_F / (||R||_F + eps) per matrix (Eq. 9-10) */
#define FIRA_FLAG_NO_SCALING 16u        /* Fira-w.o.-scaling: the factor is 1 (with gamma = inf: GaLore-add, Eq. 8) */
#define FIRA_FLAG_NO_RESIDUAL 32u       /* GaLore (Eq. 6): W <- W - lr alpha P N; the remembered norm is left alone */
/* Another base optimizer psi_t in place of Adam's Eq. 2-4 (Algorithm 2 names RMSProp, the appendix
 * reports Fira + Adagrad; the paper prints no formulas, the textbook ones are used).  M is unused.
 * The two exclude each other. */
#define FIRA_FLAG_PSI_RMSPROP 64u       /* V <- beta2 V + (1-beta2) R^2;  N = R / (sqrt V + eps) */
#define FIRA_FLAG_PSI_ADAGRAD 128u      /* V <- V + R^2;                  N = R / (sqrt V + eps) */
/* Fira-only-scaling (appendix "Theoretical Analysis", item "Variability of Scaling Factor"; the
 * only-scaling equation of the appendix on Fira versus full-rank Adam):  W <- W - lr phi(R) G.  The
 * factors k of Eq. 11 (or the one factor of Eq. 9 with FIRA_FLAG_MATRIX_SCALING) multiply the whole
 * gradient and the P N term is dropped.  Taken as Algorithm 1 with S := G diag(k): alpha and the
 * limiter act on it as they act on the scaled residual (alpha = 1 or FIRA_FLAG_ALPHA_LOWRANK_ONLY
 * together with gamma = inf give the printed equation literally).  M and V advance as usual.
 * Excludes FIRA_FLAG_NO_RESIDUAL. */
#define FIRA_FLAG_ONLY_SCALING 256u
/* Layout permission (the paper has no counterpart).  A bf16 matrix whose rows start on 16-byte
 * boundaries (ld a multiple of 8) is read and written where it is by the tensor-core kernels; if its
 * width n is not a multiple of 8 their stores, which move whole 16-byte units, also overwrite (with
 * zeros) the up to 7 padding elements that follow each row of W.  With this flag the caller allows
 * that; without it such a matrix is worked on through aligned copies in the scratch buffer (two
 * extra passes over W and one over G per step), as is every matrix whose ld is not a multiple of 8.
 * G's padding is never read or written. */
#define FIRA_FLAG_ROW_PADDING_WRITABLE 512u

/* Inputs of Algorithm 1.  eps > 0; 0 <= beta < 1; gamma >= 1 or +inf; T >= 0 (0: never). */
typedef struct {
  float beta1, beta2, eps;
  float lr;     /* eta; fira_step() can override it per call */
  float alpha;  /* GaLore scale */
  float gamma;  /* limiter threshold */
  int32_t T;    /* projection refresh gap in steps */
  uint32_t flags;
} fira_hparams;

/* One weight matrix: m x n, row major with leading dimension ld (elements, >= n;
 * 0 means n), W and G of type dtype (fira_dtype), rank 1 <= r <= min(m, n). */
typedef struct {
  int32_t m, n, r;
  int32_t dtype;
  int64_t ld;
} fira_matrix_desc;

/* Per-matrix numbers of the most recent step. */
typedef struct {
  float norm_scaled;  /* ||S|| after the column factors, before the limiter */
  float lambda;       /* limiter factor applied (1 = not limited) */
  float norm_prev;    /* ||S_prev|| now stored (norm after limiting); < 0 = unset */
  float k_min, k_max; /* range of the factors k */
  int64_t t;          /* steps taken */
  int32_t engine;     /* 0 = fp32 CUDA-core kernels, 1 = bf16 tensor-core kernels */
} fira_diag;

typedef struct fira_ctx fira_ctx;

/* Bytes needed for the state and scratch buffers of a matrix list (Algorithm 1's
 * "Input" line fixes what a matrix is; the state is the paper's comparison-table
 * count).  Both are rounded up to 256-byte multiples per section. */
FIRA_API fira_status fira_query_workspace(const fira_hparams* hp, const fira_matrix_desc* descs,
                                          int32_t count, size_t* state_bytes, size_t* scratch_bytes);

/* Algorithm 1, initialisation: M_0 = V_0 = 0, t = 0, ||S_prev|| unset, projection
 * zero (set it with fira_set_projection() or fira_refresh_projection() before the
 * first step).  state_dev and scratch_dev must be 256-byte aligned and at least as
 * large as fira_query_workspace() reports.  cuda_stream is a cudaStream_t (NULL =
 * the default stream).  Waits for the stream once the state has been cleared. */
FIRA_API fira_status fira_init(fira_ctx** out, const fira_hparams* hp, const fira_matrix_desc* descs,
                               int32_t count, void* state_dev, size_t state_bytes, void* scratch_dev,
                               size_t scratch_bytes, void* cuda_stream);

/* One pass of Algorithm 1's loop body over every matrix.  W_dev and G_dev are host
 * arrays of `count` device pointers (16-byte aligned).  W is updated in place, G is
 * only read.  lr < 0 uses hparams.lr.  With FIRA_FLAG_AUTO_REFRESH the projection of
 * every matrix whose t is a multiple of T is first recomputed from its G (the
 * "if t mod T = 0" branch). */
FIRA_API fira_status fira_step(fira_ctx* ctx, void* const* W_dev, const void* const* G_dev, float lr);

/* Plain Adam, Eq. 1-4 applied directly, for the parameters that are not projected (embeddings,
 * output head, norm gains: Section 5.1 follows GaLore's set-up, which leaves these to Adam), so
 * that a whole model can be stepped through this library:
 *   M <- b1 M + (1-b1) G;  V <- b2 V + (1-b2) G^2;  W <- W - lr sqrt(1-b2^s)/(1-b1^s) M/(sqrt V + eps)
 * with s = t + 1 (t = steps taken before this one; the caller counts).  W_dev, G_dev, M_dev, V_dev
 * are host arrays of `count` device pointers (16-byte aligned) to flat tensors of numel[i]
 * elements; W and G have type `dtype`, M and V are fp32 and owned by the caller (zero before the
 * first step).  Uses beta1, beta2, eps of hp (alpha, gamma, T and the flags do not apply); lr < 0
 * uses hp->lr.  Needs no context and no workspace.  Asynchronous on cuda_stream. */
FIRA_API fira_status fira_adam_dense(const fira_hparams* hp, int32_t count, void* const* W_dev,
                                     const void* const* G_dev, float* const* M_dev, float* const* V_dev,
                                     const int64_t* numel, fira_dtype dtype, int64_t t, float lr,
                                     void* cuda_stream);

/* The same pass as fira_step() (Algorithm 1's loop body) for callers whose weights
 * and gradients live in HOST memory: W_host and G_host are host arrays of `count`
 * host pointers (m x ld elements each; page-locked memory makes the copies
 * asynchronous).  The matrix list is cut into chunks of consecutive matrices: while
 * one chunk steps, the next one's G and W are on their way into staging_dev and the
 * previous one's W on its way back, on two copy streams that the library creates on
 * the first call and orders against the context's stream with events.  staging_dev
 * is a 256-byte aligned device buffer of at least fira_staging_bytes() bytes, owned
 * by the caller.  The host W buffers hold the result once the context's stream has
 * been synchronised.  The state after the call equals that after fira_step() on the
 * same data.  FIRA_FLAG_AUTO_REFRESH is not supported here (FIRA_ERR_UNSUPPORTED). */
FIRA_API fira_status fira_step_host(fira_ctx* ctx, void* const* W_host, const void* const* G_host,
                                    float lr, void* staging_dev, size_t staging_bytes);
FIRA_API size_t fira_staging_bytes(const fira_ctx* ctx);

/* Eq. 7: replace the projection of the selected matrices by an orthonormal basis of
 * the dominant rank-r left (m <= n) or right (m > n) singular subspace of the given
 * gradients, found on the device by `iters` rounds of blocked subspace iteration
 * started from a seeded Gaussian matrix (iters < 0: library default).  which = NULL
 * selects all matrices; G_dev always has `count` entries (entries of unselected
 * matrices may be NULL).  M, V, ||S_prev|| and t are kept.  The result spans the
 * subspace; its columns are not the individual singular vectors.  Waits for the
 * stream before returning. */
FIRA_API fira_status fira_refresh_projection(fira_ctx* ctx, const void* const* G_dev,
                                             const int32_t* which, int32_t nwhich, uint64_t seed,
                                             int32_t iters);

/* The same refresh; in addition, for every selected matrix i with basis_f32_dev[i] != NULL (a host
 * array of `count` device pointers, 16-byte aligned, d x r floats each), the basis of Eq. 7 is
 * also written there in fp32, as it stands before it is rounded to the matrix's storage type.
 * For a bf16 matrix the stored projection differs from it by one bf16 rounding per entry. */
FIRA_API fira_status fira_refresh_projection_f32(fira_ctx* ctx, const void* const* G_dev,
                                                 const int32_t* which, int32_t nwhich, uint64_t seed,
                                                 int32_t iters, float* const* basis_f32_dev);

/* Eq. 7 beside the steps (the section on gradient low-rank projection notes that the refresh costs
 * little when it runs only every T steps; this entry point takes it off the step's stream altogether).  The
 * same iteration as fira_refresh_projection(), but nothing of the context is modified: it works in
 * work_dev (256-byte aligned, at least fira_refresh_side_work_bytes() bytes: room for the largest
 * matrix; more room lets it take several matrices per pass), enqueues on side_stream (a cudaStream_t
 * other than the context's) and writes the basis of every selected matrix i to P_out_dev[i] (a host
 * array of `count` device pointers, d x r in the matrix's dtype, 16-byte aligned).  The call may be
 * made from another host thread while fira_step() runs on the context's stream (it reads only what
 * fira_init() fixed); it waits for side_stream before returning.  To adopt a basis, order the
 * context's stream after side_stream and call fira_set_projection().  Same seed, same gradients:
 * the same bases as fira_refresh_projection(), bit for bit. */
FIRA_API size_t fira_refresh_side_work_bytes(const fira_ctx* ctx);
FIRA_API fira_status fira_refresh_projection_side(fira_ctx* ctx, const void* const* G_dev,
                                                  const int32_t* which, int32_t nwhich, uint64_t seed,
                                                  int32_t iters, void* const* P_out_dev, void* work_dev,
                                                  size_t work_bytes, void* side_stream);

/* Copy a projection (d x r, row major, the matrix's dtype) from / to device memory
 * (the P_t of Algorithm 1, given by the caller instead of Eq. 7). */
FIRA_API fira_status fira_set_projection(fira_ctx* ctx, int32_t idx, const void* P_dev);
FIRA_API fira_status fira_get_projection(fira_ctx* ctx, int32_t idx, void* P_dev);

/* Checkpointing of Algorithm 1's state: copy M and V (l x r floats each, device
 * pointers, may be NULL to skip) and the two scalars.  Both wait for the stream. */
FIRA_API fira_status fira_get_state(fira_ctx* ctx, int32_t idx, float* M_dev, float* V_dev,
                                    float* norm_prev_host, int64_t* t_host);
FIRA_API fira_status fira_set_state(fira_ctx* ctx, int32_t idx, const float* M_dev, const float* V_dev,
                                    float norm_prev, int64_t t);

/* Number of optimizer-state elements held for matrix idx: d r + 2 l r + 1 (the
 * "Optimizer States" row of the paper's comparison table). */
FIRA_API int64_t fira_state_elements(const fira_ctx* ctx, int32_t idx);

/* Waits for the stream and copies the diagnostics of matrix idx (the quantities of
 * Eq. 11 and Eq. 12 of the latest step) to the host. */
FIRA_API fira_status fira_get_diagnostics(fira_ctx* ctx, int32_t idx, fira_diag* out_host);

/* Reads the device status word (waits for the stream): FIRA_OK, or the first
 * device-side condition recorded since the last poll, which it clears. */
FIRA_API fira_status fira_poll(fira_ctx* ctx);

/* Self-test of the failure path of the tensor-core kernels (the paper has no counterpart).  Every
 * wait inside those kernels is bounded: a wait that runs out raises a flag that all roles of the
 * block poll, the kernel returns, and the time-out shows up in fira_poll().  This call enqueues a
 * one-block kernel whose waits can never be satisfied (a barrier that nothing arrives on, no copy in
 * flight; a counter in global memory that nothing raises, the form in which the projection epilogues
 * wait for one another) with a limit of `rounds` tries (1 .. 2^20), so that the path can be exercised without
 * disturbing anything: afterwards fira_poll() returns FIRA_ERR_DEVICE_TIMEOUT once, then FIRA_OK,
 * and the context steps on as before. */
FIRA_API fira_status fira_selftest_bounded_wait(fira_ctx* ctx, int32_t rounds);

/* Number of kernel launches enqueued by the most recent fira_step() call. */
FIRA_API int32_t fira_last_step_launches(const fira_ctx* ctx);

/* Per-kernel timing of fira_step() (measurement aid; the paper has no counterpart).
 * While enabled, every step records CUDA events on the context's stream before and
 * after each of its kernels (the last FIRA_TIMING_MAX_STEPS steps are kept).
 * fira_get_phase_times() waits for the stream and returns, per kernel ("phase") in
 * launch order, the mean duration in milliseconds over the recorded steps; ms_out
 * has room for FIRA_TIMING_MAX_PHASES floats.  fira_phase_name() names a phase. */
#define FIRA_TIMING_MAX_PHASES 16
#define FIRA_TIMING_MAX_STEPS 64
FIRA_API fira_status fira_enable_phase_timing(fira_ctx* ctx, int32_t enable);
FIRA_API fira_status fira_get_phase_times(fira_ctx* ctx, int32_t* nphases, float* ms_out,
                                          int32_t* steps_recorded);
FIRA_API const char* fira_phase_name(const fira_ctx* ctx, int32_t phase);

/* One step of ONE matrix without any buffer from the caller beyond the inputs and
 * outputs themselves.  (The paper has no counterpart: this is a deployment aid.)
 *
 * It exists for callers that are not allowed to allocate device memory -- code
 * running inside another framework's memory pool, a latency-critical loop that must
 * stay out of the driver's allocator, a process whose memory was budgeted at start
 * -- and therefore cannot provide the state and scratch buffers of fira_init().  The
 * intermediates live in a fixed array inside the library image instead:
 * fira_noalloc_max_scratch_bytes() bytes (8 MiB), held on every GPU that loads the
 * library until the process exits.  The call allocates nothing.
 *
 * desc: the matrix (fp32 or bf16; it always runs on the fp32 CUDA-core kernels).  Its
 * intermediates must fit the array, roughly max(m,n) * r <= 1,000,000; larger
 * matrices are rejected with FIRA_ERR_WORKSPACE_TOO_SMALL and a message giving the
 * sizes.  W_dev (updated in place), G_dev, P_dev (the d x r projection), M_dev and
 * V_dev (l x r floats, zero before the first step, updated in place) are 16-byte
 * aligned device pointers; norm_prev_dev points to one float on the device (set it
 * to -1 before the first step: "no remembered norm yet") and t_dev to one int64 on
 * the device (0 before the first step); both are updated.  lr < 0 uses hp->lr.
 * The result equals fira_step()'s for the same matrix on the CUDA-core kernels.
 *
 * Host-side argument errors (including the variant flags, none of which this entry
 * point supports: FIRA_ERR_UNSUPPORTED) are returned before anything is enqueued.
 * Device-side conditions (a non-finite norm) are recorded in a status word inside the
 * array; fira_noalloc_poll() waits for the given stream, returns FIRA_OK or the
 * condition, and clears it (it allocates nothing either).
 *
 * The first call on a device looks up the array's device address (host threads may
 * race to it: the look-up is serialised); make that call before any stream capture
 * starts.  All calls share the one array, which keeps the previous call's contents
 * (each call rewrites what it reads), so calls that overlap on the GPU -- from
 * different streams or threads -- race: issue them on one stream or wait in between. */
FIRA_API fira_status fira_step_single_noalloc(const fira_hparams* hp, const fira_matrix_desc* desc,
                                              void* W_dev, const void* G_dev, const void* P_dev,
                                              float* M_dev, float* V_dev, float* norm_prev_dev,
                                              int64_t* t_dev, float lr, void* cuda_stream);
FIRA_API size_t fira_noalloc_max_scratch_bytes(void);
FIRA_API fira_status fira_noalloc_poll(void* cuda_stream);

FIRA_API const char* fira_status_string(fira_status s);
/* Text of the most recent error on this thread ("" if none). */
FIRA_API const char* fira_last_error(void);
FIRA_API void fira_destroy(fira_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FIRA_H_ */
