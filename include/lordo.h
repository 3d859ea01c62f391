/*
 * lordo.h -- C ABI of the LoRDO optimizer hot path on one NVIDIA B200 (sm_100a).
 *
 * The library runs, for a list of weight matrices W_i (m_i x n_i) and K simulated workers held as
 * a replica axis on one GPU, the three recurring pieces of the paper's Algorithm 1 (Global
 * variant) and Algorithm 2 (Local variant):
 *
 *   lordo_inner_step       the per-step block: clip, project with error feedback, low-rank Adam
 *                          moments, (quasi-hyperbolic) update, back-projection onto W
 *   lordo_outer_step       the synchronisation block: state averaging, pseudo-gradient mean,
 *                          outer optimizer (averaging or Nesterov), broadcast
 *   lordo_refresh_subspace ComputeProjection (randomized range finder + QR) and the rotation of
 *                          the moments into the new basis
 *   lordo_init             the algorithms' "Require" block (initial P, zero states, anchor copy)
 *
 * Conventions
 *   - Every matrix is row-major with no padding. The replica axis is outermost and contiguous:
 *     W_i is [K][m][n]; u_i, v_i are [K][r][n]; P_i is [m][r] (Global) or [K][m][r] (Local).
 *   - All "device" pointers are CUDA device memory of the current device, owned by the caller,
 *     16-byte aligned, and must stay valid for the lifetime of the context. The library never
 *     allocates device memory; `workspace` (size from lordo_query_workspace) is caller-owned too.
 *   - Pointer *tables* (`void* const*`) are host arrays with one device pointer per matrix.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream). Calls enqueue work
 *     and return without synchronising, except lordo_init, lordo_poll_status,
 *     lordo_inner_step_host, lordo_profile_read and lordo_destroy. (A call that is handed new
 *     gradient pointers stages their table in one of two pinned slots and may wait for the copy
 *     that left that slot two changes ago, which has normally long finished.)
 *   - Shapes: n and r multiples of 8 (m too for a matrix projected from the right), 8 <= r <= min(m, n),
 *     K >= 1, H >= 1.
 *   - Errors are return codes (lordo_status); nothing throws or aborts. After a non-zero return
 *     from an argument check no device state was modified. Numerical trouble found on the device
 *     (non-finite gradient norm, breakdown of the QR) sets a sticky flag word that
 *     lordo_poll_status returns.
 *   - A context is not thread-safe. Call order is checked (LORDO_ERR_STATE): lordo_outer_step
 *     only after a multiple of H inner steps; Global lordo_refresh_subspace only directly after
 *     lordo_outer_step; Local lordo_refresh_subspace only before the first inner step of a round.
 */
#ifndef LORDO_H_
#define LORDO_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LORDO_API __attribute__((visibility("default")))
#else
#define LORDO_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lordo_ctx lordo_ctx; /* opaque, host memory, library-owned */

typedef enum {
  LORDO_OK = 0,
  LORDO_ERR_INVALID_ARG = 1,
  LORDO_ERR_SHAPE = 2,
  LORDO_ERR_ALIGN = 3,
  LORDO_ERR_STATE = 4,
  LORDO_ERR_NOMEM = 5,
  LORDO_ERR_CUDA = 6,
  LORDO_ERR_NUMERIC = 7,
  LORDO_ERR_UNSUPPORTED = 8
} lordo_status;

typedef enum { LORDO_F32 = 0, LORDO_BF16 = 1 } lordo_dtype;
typedef enum { LORDO_GLOBAL = 0, LORDO_LOCAL = 1 } lordo_variant;                 /* Alg. 1 / Alg. 2 */
typedef enum { LORDO_QHM_NONE = 0, LORDO_QHM_LOW = 1, LORDO_QHM_FULL = 2 } lordo_qhm; /* Alg. 1, update cases */
typedef enum { LORDO_OUTER_AVG = 0, LORDO_OUTER_NESTEROV = 1 } lordo_outer;       /* OuterOpt */

/* device status flags returned by lordo_poll_status */
#define LORDO_FLAG_NONFINITE_GRAD 1u /* a gradient norm was NaN or Inf */
#define LORDO_FLAG_QR_BREAKDOWN 2u   /* a column of a sketch was (numerically) dependent on the columns before it */
#define LORDO_FLAG_DEVICE_TIMEOUT 4u /* a bounded wait inside a kernel gave up; results of that call are invalid */

typedef struct {
  int64_t m, n; /* W is m x n */
  int32_t r;    /* P is m x r; moments are r x n (projection from the left, Sec. 2) */
  int32_t side; /* 0: as in the paper, from the left. 1: from the right (not in the paper, which always projects
                   from the left; the side selection of GaLore-type methods for matrices with m > n): P is n x r,
                   g = (G^ + E) P, the update is U~ P^T, mu(.) of the full-rank QHM term gives one value per row,
                   ComputeProjection returns the top-r right singular subspace. It is the left-side method applied
                   to W^T, and the library keeps that view: the moments u, v of such a matrix are [K][r][m]
                   (transposed low-rank arrays), P is [n][r] / [K][n][r]. Needs m a multiple of 8; not available
                   together with time_buffer or oversample. */
} lordo_mat;

typedef struct {
  int32_t n_mats;
  const lordo_mat* mats;   /* host array [n_mats] */
  int32_t K;               /* workers held as replicas (paper: M) */
  int32_t H;               /* inner steps per round (paper: K_x = K_u = K_v) */
  int32_t w_dtype;         /* lordo_dtype of W */
  int32_t g_dtype;         /* lordo_dtype of the gradients */
  int32_t e_dtype;         /* lordo_dtype of the error buffer E */
  int32_t variant;         /* lordo_variant */
  int32_t error_feedback;  /* 1: g = P^T(G^ + E), E <- G^ + E - P g ; 0: g = P^T G^, E unused */
  float beta2;             /* second-moment decay */
  float eps;               /* Adam epsilon */
  float clip_rho;          /* clipping radius rho; <= 0 disables clipping */
  int32_t clip_scope;      /* 0: one norm per worker over all matrices; 1: one per matrix */
  int32_t sync_u, sync_v;  /* average u / v over workers in lordo_outer_step */
  int32_t outer;           /* lordo_outer */
  float outer_lr;          /* eta_s (Nesterov only) */
  float outer_momentum;    /* mu_s  (Nesterov only) */
  int32_t power_iters;     /* subspace iterations of the range finder (0..8) */
  uint64_t seed;           /* seed of the counter-based generator for P_0 and the sketches */
  int32_t check_mode;      /* 1: every contraction in fp32 FMA arithmetic (parity mode);
                              0: bf16 tensor-core contractions where operands are bf16 */
  int32_t warm_start;      /* 0: every refresh starts from a fresh random sketch; 1: block power iteration
                              started from the current P (max(power_iters, 1) iterations, no sketch), the
                              cheaper estimator the paper names as an alternative ComputeProjection */
  int32_t time_buffer;     /* 1: the up-link time buffer of App. "Worker Communication": every worker accumulates
                              T += eta * alpha (alpha = the step's low-rank update, r x n, workspace memory) and
                              lordo_outer_step rebuilds the pseudo-gradient as (1/K) sum_k P_k T_k instead of
                              reading it off the K weight replicas. Only the update forms without the full-rank
                              term factorise: lordo_inner_step with LORDO_QHM_FULL returns LORDO_ERR_UNSUPPORTED.
                              The basis does not move between two synchronisations (the call order that
                              lordo_refresh_subspace enforces), which the factorisation needs. 0: off */
  int32_t oversample;      /* p >= 0, a multiple of 8: the range finder of the refresh runs with r + p columns and its
                              basis is truncated to the top-r left singular subspace of its projection of the
                              signal (Rayleigh-Ritz; not in the paper, the randomized-SVD refinement of the range
                              finder). The refresh then runs in fp32 in both modes. Needs r + p <= min(m, n) and
                              <= 600 for every matrix and warm_start = 0. 0: off */
} lordo_config;

/* Host tables of device pointers, one entry per matrix. fp32 unless stated. */
typedef struct {
  void* const* W;      /* [K][m][n] in w_dtype; on entry to lordo_init replica 0 holds W_0 */
  void* const* E;      /* [K][m][n] in e_dtype; may be NULL when error_feedback == 0 */
  float* const* P;     /* [m][r] (Global) or [K][m][r] (Local); side 1: [n][r] / [K][n][r] */
  float* const* u;     /* [K][r][n] first moment; side 1: [K][r][m] */
  float* const* v;     /* [K][r][n] second moment; side 1: [K][r][m] */
  float* const* X0;    /* [m][n] model copy of the last synchronisation */
  float* const* B;     /* [m][n] outer momentum; may be NULL when outer == LORDO_OUTER_AVG */
  float* const* Delta; /* [m][n] aggregated pseudo-gradient of the last lordo_outer_step */
} lordo_buffers;

/* Bytes of device workspace lordo_init needs for this configuration. Host-only, no CUDA call. */
LORDO_API int lordo_query_workspace(const lordo_config* cfg, size_t* bytes);

/*
 * Algorithm 1 / 2 "Require": copies W[0] to every replica and to X0, zeroes E, u, v, B, Delta,
 * writes P_0 (Global: orthonormalised random matrix from `seed`; Local: first r columns of the
 * identity for every worker). Synchronises `stream` before returning. `*out` owns host memory
 * only and is released by lordo_destroy. `workspace` must be 256-byte aligned.
 */
LORDO_API int lordo_init(const lordo_config* cfg, const lordo_buffers* buf, void* workspace, size_t workspace_bytes,
               void* stream, lordo_ctx** out);

/*
 * Algorithm 1, the per-step lines (clip ... model update), for every matrix and worker.
 * G: host table of device pointers, G[i] is [K][m_i][n_i] in g_dtype, read only.
 * lr = eta_t; beta1, omega per call because the paper switches them after warm-up; form selects
 * the update case. Bias correction uses the count of inner steps done on this context.
 */
LORDO_API int lordo_inner_step(lordo_ctx* ctx, const void* const* G, float lr, float beta1, float omega, int form,
                     void* stream);

/*
 * Same step fed from HOST memory: copies G_host[i] (pinned or pageable host memory, [K][m][n] in
 * g_dtype) into the caller's device staging buffers G_stage[i], runs lordo_inner_step, copies the
 * K clip coefficients of matrix 0 back to clip_out_host (K floats, may be NULL) and synchronises.
 */
LORDO_API int lordo_inner_step_host(lordo_ctx* ctx, const void* const* G_host, void* const* G_stage, float lr, float beta1,
                          float omega, int form, float* clip_out_host, void* stream);

/*
 * Algorithm 1, synchronisation lines: u,v <- mean over workers (if sync_u / sync_v);
 * Delta = X0 - mean_k W_k; averaging: X0 <- X0 - Delta; Nesterov: B <- mu_s B + Delta,
 * X0 <- X0 - eta_s (Delta + mu_s B); every W_k <- X0.
 */
LORDO_API int lordo_outer_step(lordo_ctx* ctx, void* stream);

/*
 * Algorithm 1, lines "if t mod K_u = 0: u <- E_m[u]" and "if t mod K_v = 0: v <- E_m[v]" on their
 * own, for schedules whose state-synchronisation intervals K_u, K_v differ from the model interval
 * K_x = H (set sync_u = sync_v = 0 in the configuration and call this at the steps of your choice).
 * May be called between any two inner steps.
 */
LORDO_API int lordo_sync_states(lordo_ctx* ctx, int sync_u, int sync_v, void* stream);

/*
 * ComputeProjection and the moment-rotation lines of Algorithm 1 (Global: signal = Delta, G must
 * be NULL) or Algorithm 2 (Local: signal = c_k G_k + E_k per worker, G as for lordo_inner_step).
 * Range finder: Y = S Omega with an n x r integer sketch from `seed`, thin QR, `power_iters`
 * subspace iterations. If at least one inner step was done the moments are rotated with
 * Rot = P_new^T P_old: u <- Rot u, v <- (1-beta2^s)|(Rot o Rot)(v^ - u^ o u^) + (Rot u^) o (Rot u^)|.
 * beta1 is the first-moment decay used for the bias-corrected u^.
 */
LORDO_API int lordo_refresh_subspace(lordo_ctx* ctx, const void* const* G_or_null, float beta1, void* stream);

/* Synchronises `stream`, stores the sticky device flag word in *flags (may be NULL) and returns
 * LORDO_ERR_NUMERIC if it is non-zero, else LORDO_OK. */
LORDO_API int lordo_poll_status(lordo_ctx* ctx, void* stream, uint32_t* flags);

/*
 * Diagnostics (Sec. "Experimental Framework", Metrics). mssv_dev: one float per projection matrix
 * (n_mats for Global, n_mats * K for Local, matrix-major), the mean squared singular value
 * (1/r) sum_i sigma_i^2 of Rot = P_new^T P_old of the LAST lordo_refresh_subspace (1 = the subspace
 * did not move, 0 = it moved to an orthogonal one); valid until the next refresh overwrites the
 * rotation matrices; LORDO_ERR_STATE before the first refresh. e_norm_dev: [n_mats][K] floats,
 * ||E||_F of every error buffer. Either pointer may be NULL. Device pointers, caller-owned.
 */
LORDO_API int lordo_diagnostics(lordo_ctx* ctx, float* mssv_dev, float* e_norm_dev, void* stream);

/* Clears the sticky device flag word (after the caller has dealt with what lordo_poll_status reported). */
LORDO_API int lordo_clear_status(lordo_ctx* ctx, void* stream);

/*
 * Self-test of the failure path of the tensor-core kernels: every wait inside them (on a TMA
 * transfer, a tensor-core commit, another warp) is bounded; a wait that runs out sets
 * LORDO_FLAG_DEVICE_TIMEOUT and the kernel runs to its normal end, so the context stays usable.
 * This call enqueues a one-thread kernel that waits on a barrier nothing completes: about two
 * seconds later lordo_poll_status reports the flag. It touches no optimizer state.
 */
LORDO_API int lordo_selftest_wait_timeout(lordo_ctx* ctx, void* stream);

/* Counters for checkpoint / resume: {inner steps done, refreshes done, outer steps done, inner steps
 * done in the current round}. A checkpoint is the caller's tensors (W, E, P, u, v, X0, B, Delta) plus
 * these four numbers: restore the tensors into the buffers of a context made with the same
 * configuration, then call lordo_set_counters (which also makes the library rebuild its internal
 * copies of P before the next step). With time_buffer the low-rank accumulators of a round live in the
 * workspace and are not part of a checkpoint: lordo_set_counters then accepts round boundaries only
 * (in[3] == 0, where the accumulators are zero) and returns LORDO_ERR_UNSUPPORTED otherwise.
 * Global rule: a checkpoint taken between lordo_outer_step and lordo_refresh_subspace (a round boundary
 * with fewer refreshes than synchronisations) may run that refresh first thing after the restore. The
 * rotation matrices behind lordo_diagnostics' MSSV are workspace state too: after a restore MSSV returns
 * LORDO_ERR_STATE until a refresh has run on the new context. */
LORDO_API int lordo_get_counters(const lordo_ctx* ctx, int64_t out[4]);
LORDO_API int lordo_set_counters(lordo_ctx* ctx, const int64_t in[4]);

/* Device address of the clip coefficients of the last inner step, [n_mats][K] fp32 (library
 * workspace; valid until lordo_destroy). */
LORDO_API int lordo_clip_coefficients(const lordo_ctx* ctx, const float** device_ptr);

/* Number of kernels this context has launched so far. */
LORDO_API int64_t lordo_launch_count(const lordo_ctx* ctx);

/*
 * Per-kernel-class device timing with CUDA events on the call's stream. While enabled, every
 * call records an event pair around each class; lordo_profile_read synchronises `stream` and
 * returns the milliseconds accumulated since the previous read:
 * ms[0] clip norm, [1] projection g = P^T(cG+E), [2] moment update, [3] back-projection + weight
 * and error-buffer update, [4] state averaging, [5] outer update, [6] subspace refresh, [7] unused.
 */
LORDO_API int lordo_profile_enable(lordo_ctx* ctx, int on);
LORDO_API int lordo_profile_read(lordo_ctx* ctx, void* stream, float ms_out[8]);

/* Text of the last error of this context (library-owned, valid until the next call). */
LORDO_API const char* lordo_last_error(const lordo_ctx* ctx);
LORDO_API const char* lordo_status_string(int status);

LORDO_API int lordo_destroy(lordo_ctx* ctx);

/*
 * The counter-based generator behind P_0 and the sketches, exposed so that it can be compared
 * bit for bit with a host implementation: out[i*cols + j] = popcount(mix64(key + g*(i*cols+j+1))) - 32
 * with key chained from (seed, purpose, mat, index, replica); purpose 1 = P_0, 2 = sketch.
 * out_dev: device pointer, rows*cols floats.
 */
LORDO_API int lordo_fill_random(uint64_t seed, int32_t purpose, int32_t mat, int64_t index, int32_t replica, int64_t rows,
                      int64_t cols, float* out_dev, void* stream);

/*
 * (The paper has no counterpart for this entry point; it is a convenience of this library.)
 *
 * Clip coefficient c = min(1, rho / (||G||_2 + 1e-6)) of ONE gradient array, computed without any
 * device allocation: no context, no workspace. It is meant for callers that must not or cannot
 * allocate device memory at the point where they need the coefficient -- code running while a
 * memory pool is frozen or nearly exhausted, a plug-in that was handed fixed buffers by its host
 * framework, a monitoring hook that may not disturb the allocator of the job it watches.
 * The reduction's partial sums live in a fixed array inside the library image (128 KiB per GPU
 * that loads the library, held until the process exits), which bounds the input:
 * count <= lordo_clip_coefficient_static_max_count() (2^29 elements); larger inputs are rejected
 * with LORDO_ERR_UNSUPPORTED and nothing is launched.
 *
 *   G_dev         device pointer, `count` elements of g_dtype (lordo_dtype), 16-byte aligned,
 *                 count a multiple of 8; read only
 *   rho           clipping radius; <= 0 gives c = 1
 *   coef_out_dev  device pointer to one float, written by the call (caller-owned); NaN when the
 *                 sum of squares is NaN or infinite (this entry point has no status word)
 *
 * The call enqueues two kernels on `stream` and returns without synchronising. The first call on
 * each device looks up the device address of the static array (with that device current); make
 * that first call outside any stream capture (the address is cached for the life of the process
 * and does not survive a cudaDeviceReset). A CUDA error already pending on the thread makes the
 * call return LORDO_ERR_CUDA before it launches anything. All calls on a device share the array: it holds
 * whatever the previous call left (every slot a call reads it has written itself, so nothing needs
 * clearing), and two calls whose kernels overlap on the GPU -- different streams, no ordering
 * between them -- race on it. Calls on one stream are safe.
 */
LORDO_API int lordo_clip_coefficient_static(const void* G_dev, int g_dtype, int64_t count, float rho, float* coef_out_dev,
                                            void* stream);
LORDO_API int64_t lordo_clip_coefficient_static_max_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LORDO_H_ */
