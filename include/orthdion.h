/* orthdion.h - C interface of the B200 (sm_100a) Orth-Dion / Dion optimizer-step library.
 *
 * One call of orthdion_step advances one weight matrix by one step of the paper's Algorithm 1
 * (the one-step statement of Orth-Dion and of Dion with its auxiliary machinery stripped; the
 * appendix gives both as full loops).  The library runs it as five stages, written here with the
 * letters of this interface (the paper's letters in brackets):
 *
 *   K1     Y = (M + G) * Q_prev        the buffer B = M + G [M_t = G_t + R_t] is formed on the
 *                                      fly and never stored; Q_prev is the carried right
 *                                      factor [V_{t-1}]
 *   QR     P = orth(Y)                 left factor [U_t]
 *   K3     R = (M + G)^T * P           un-normalised right factor [W_t]
 *   QR or  Q = orth(R)   (ORTH)        Orth-Dion's normalisation of the right factor, or
 *   scale  Q = ColNorm(R) (COLNORM)    Dion's unit-length columns [V_t]
 *   K5     X <- (1 - eta*wd) * X - eta*scale * P * Q^T      weight update, and in the same pass
 *          M <- a * (M + G) - b * P * R^T                   the error-feedback residual [R_{t+1}]
 *
 * Q then serves as Q_prev of the next step.  orth(.) is the thin QR factor with a positive
 * diagonal in the triangular factor (CholeskyQR2 on the device, with a shifted third pass when
 * the Gram matrix is ill-conditioned).  (a, b) default to (1, 1 - mu); the paper's own residual
 * rule is (beta, beta).
 *
 * Conventions
 *  - Every matrix pointer is a DEVICE pointer owned by the caller; matrices are row-major and
 *    contiguous: X, M, G are m x n (leading dimension n), Q is n x r (leading dimension r).
 *  - X, M and Q are updated in place; G is only read.  Q holds Q_prev on entry, Q on return.
 *  - M and Q are float32.  X and G are float32 or bfloat16 (orthdion_set_dtypes).
 *  - All device pointers must be 16-byte aligned.
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *    synchronising.  The device that owns `stream` and the matrices must be the current device
 *    of the calling thread; per-device set-up (kernel attributes, internal streams) is keyed by
 *    it.  The library allocates no device memory: the caller passes a workspace of at least
 *    orthdion_workspace_bytes*() bytes, 256-byte aligned, which must stay untouched until the
 *    enqueued work has finished.  P, R, the status words and the diagnostic records live in it.
 *  - Return value: 0 on success, a negative ORTHDION_ERR_* code when the host rejects the
 *    arguments (nothing is enqueued then).  Numerical conditions never trap: they are reported
 *    per matrix through status flags in the workspace (orthdion_last_status).  A matrix whose
 *    factorisation fails even after the shifted pass keeps X, M and Q unchanged.
 *  - Handles are immutable plans apart from the setters and may be shared by any number of
 *    matrices of the same shape.  Setters must not race with a step call on the same handle.
 *  - The library needs a CUDA device of compute capability 10.x; there is no CPU fallback.
 */
#ifndef ORTHDION_H_
#define ORTHDION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct orthdion_plan* orthdion_t;

/* Algorithm 1, normalisation step: which normalisation of the right factor. */
#define ORTHDION_MODE_ORTH     0   /* Q = orth(R): Orth-Dion                     */
#define ORTHDION_MODE_COLNORM  1   /* Q = ColNorm(R): (Stripped) Dion            */

#define ORTHDION_DTYPE_F32   0
#define ORTHDION_DTYPE_BF16  1

/* Which kernels carry the matrix products.  TENSOR: tcgen05 tensor-core kernels with
 * bf16-split operands and fp32 accumulation in tensor memory.  SIMT: plain fp32 FMA kernels
 * (any r >= 1; meant for tiny matrices and as an on-device cross-check). */
#define ORTHDION_ENGINE_TENSOR 0
#define ORTHDION_ENGINE_SIMT   1

/* host-side error codes */
#define ORTHDION_OK                 0
#define ORTHDION_ERR_INVALID_ARG   -1   /* bad handle, count, mode, dtype, engine, scalar       */
#define ORTHDION_ERR_RANK          -2   /* r < 1, r > min(m, n), or r not supported by engine   */
#define ORTHDION_ERR_NULL          -3   /* a required pointer is null                           */
#define ORTHDION_ERR_WORKSPACE     -4   /* workspace too small or misaligned                    */
#define ORTHDION_ERR_CUDA          -5   /* a CUDA runtime call failed (launch, attribute, ...)  */
#define ORTHDION_ERR_ALIGNMENT     -6   /* a matrix pointer is not 16-byte aligned              */

/* per-matrix device status flags (bit mask) */
#define ORTHDION_STATUS_SHIFTED_LEFT    1   /* left QR took three passes (shifted first pass,   */
#define ORTHDION_STATUS_SHIFTED_RIGHT   2   /* or a second pass that met a poorly conditioned   */
                                            /* Q1); same for the right QR                       */
#define ORTHDION_STATUS_RANK_DEFICIENT  4   /* factorisation failed: X, M, Q left unchanged     */
#define ORTHDION_STATUS_NONFINITE       8   /* a Gram matrix held Inf/NaN: treated as failure   */
#define ORTHDION_STATUS_ZERO_COLUMN    16   /* COLNORM met a zero column of R (kept zero)       */
#define ORTHDION_STATUS_WAIT_LIMIT     32   /* a bounded device-side wait expired (kernel bug): */
                                            /* set on every matrix of the launch; M and X of    */
                                            /* those matrices may be partially updated          */

/* Create a plan for m x n matrices at rank r (inputs of Algorithm 1: step size eta, EF
 * coefficient; mu gives the default (a, b) = (1, 1 - mu)).  Defaults: X and G bfloat16,
 * scale = 1, engine TENSOR.  The TENSOR engine needs r % 16 == 0, n % 8 == 0 and takes
 * r <= 4096 (the rank fraction 0.25 of the paper's 16384-wide blocks); SIMT takes any
 * r <= 1024 and is chosen when the TENSOR conditions do not hold.  Diagnostics need r <= 1024.
 * ORTHDION_ERR_RANK otherwise.  Host memory only. */
int orthdion_create(orthdion_t* out, int64_t m, int64_t n, int32_t r,
                    float mu, float eta, float wd, int32_t mode);
int orthdion_destroy(orthdion_t h);

int orthdion_set_dtypes(orthdion_t h, int32_t x_dtype, int32_t g_dtype);
int orthdion_set_lr(orthdion_t h, float eta);               /* eta_t of a schedule               */
int orthdion_set_scale(orthdion_t h, float scale);          /* extra factor on the update; 1.0   */
int orthdion_set_ef(orthdion_t h, float a, float b);        /* M <- a*B - b*P*R^T                */
int orthdion_set_engine(orthdion_t h, int32_t engine);
/* Number of tensor-core passes products are built from (3 = three bf16 products of a two-term
 * split, about 2^-16 relative accuracy; 1 = one pass).  which: 0 = B*Q and B^T*P, 1 = Gram/apply
 * of the QR, 2 = P*R^T of the error feedback, 3 = P*Q^T of the weight update.  When both 2 and 3
 * ask for one pass, the fused pass runs in fp16 (11-bit operands, R scaled by a power of two);
 * otherwise a single pass means plain bf16.  Defaults: 3 and 3; for the fused pass 1, 1 with bf16
 * weights while |b| <= 0.1 |a| (the momentum form), 3, 1 with bf16 weights otherwise (in the
 * residual form a = b the fp16 error of P*R^T, about 4e-4, would show in M), 3, 3 with fp32
 * weights.  The defaults follow later calls of set_dtypes and set_ef until a count is set here;
 * passes <= 0 hands it back to the default rule. */
int orthdion_set_passes(orthdion_t h, int32_t which, int32_t passes);

/* Workspace sizes in bytes (host computation, no CUDA call). */
size_t orthdion_workspace_bytes(orthdion_t h);
size_t orthdion_workspace_bytes_grouped(const orthdion_t* hs, int32_t count);

/* One step for one matrix (Algorithm 1). */
int orthdion_step(orthdion_t h, void* X, float* M, const void* G, float* Q,
                  void* workspace, size_t workspace_bytes, void* stream);

/* One step for `count` matrices; hs[i] is the plan of matrix i.  X, M, G, Q are HOST arrays of
 * `count` device pointers.  Matrices with equal plan parameters are sorted into packs and every
 * stage runs once per pack (the batching of equal shapes that the paper's appendix on its
 * wide-model study mentions).  Results per matrix are identical to orthdion_step.
 * The call may be recorded into a CUDA graph by stream capture on `stream` and replayed (the
 * pointers and plan settings are baked into the graph): make one call on the device outside the
 * capture first, which sets kernel attributes and creates the internal streams. */
int orthdion_step_grouped(const orthdion_t* hs, int32_t count,
                          void* const* X, float* const* M, const void* const* G, float* const* Q,
                          void* workspace, size_t workspace_bytes, void* stream);

/* How many launch batches (matrices of equal plan) a grouped call may step side by side.  The
 * optimizer steps of two matrices are independent (nothing in Algorithm 1 couples them), so the
 * grouped call forks the caller's stream into `lanes` internal streams, runs every batch's
 * stage sequence on one of them and joins them again before it returns: everything enqueued on
 * `stream` after the call still waits for the whole step, and the host never blocks.  Results per
 * matrix are bit for bit those of lanes = 1.  1 <= lanes <= 8; default 4.  Process-wide; the first
 * grouped call on a device creates that device's internal streams and events (no device memory);
 * two grouped calls on the same device are serialised on the host while they enqueue. */
int orthdion_set_concurrency(int32_t lanes);

/* Column-sharded step: one weight matrix split by columns over k ranks (the paper's FSDP setting,
 * Section 2, "FSDP communication": only O((m + n) r) numbers cross the ranks per step).  Rank j
 * holds X_j, M_j, G_j (m x n_j, its columns) and Q_j (n_j x r, the matching rows of the right
 * factor); its plan is created with (m, n_j, r).  Since B Q_prev = sum_j B_j Q_j, R_j = B_j^T P and
 * R^T R = sum_j R_j^T R_j, the step is a sequence of local phases with one sum over the ranks of a
 * small fp32 buffer between two phases.  The caller makes that sum (an all-reduce on real ranks)
 * in place on the buffer that orthdion_shard_reduce_buffer returns for the phase just run, then
 * runs the next phase:
 *   phase 0   Y_j = (M_j + G_j) Q_j                        reduce: Y, m x r
 *   phase 1   P = orth(Y), the same on every rank; R_j = (M_j + G_j)^T P;
 *             ORTH: Gram matrix of R_j                      reduce: r x r  (entries above the
 *                                                           256 x 256 diagonal tiles are not used)
 *             COLNORM: squared column norms of R_j          reduce: r
 *   phase 2   ORTH: first CholeskyQR pass of R_j with the summed Gram matrix, Gram matrix of the
 *             result                                        reduce: r x r
 *             COLNORM: Q_j = R_j / norms; X_j, M_j updated: the step is complete
 *   phase 3   ORTH only: second pass, Q_j; X_j, M_j updated: the step is complete
 * Every phase is enqueued on `stream`; the same workspace (orthdion_workspace_bytes of the plan)
 * must be passed to all phases of a step and keeps P, R_j and the status word afterwards
 * (orthdion_get_factors, orthdion_last_status with count 1).  TENSOR engine only, diagnostics
 * off.  The right QR is CholeskyQR2 here: a third pass that the second one asks for
 * (ORTHDION_STATUS_SHIFTED_RIGHT) is reported but not taken.  With one shard and no reduction the
 * phases compute what orthdion_step computes. */
int orthdion_shard_phase(orthdion_t h, int32_t phase, void* X, float* M, const void* G, float* Q,
                         void* workspace, size_t workspace_bytes, void* stream);
/* Device pointer and length (in floats) of the buffer to sum over the ranks after `phase`. */
int orthdion_shard_reduce_buffer(orthdion_t h, int32_t phase, void* workspace, float** buffer, int64_t* count);

/* One step for one matrix without any caller-provided workspace and without any device-memory
 * allocation.  (The paper has no counterpart: this entry point exists for the integration, not
 * for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region that is being
 * stream-captured, inside a framework callback that must not touch the allocator, or in a process
 * whose memory pool was sized up front and locked.  Such a caller cannot size and allocate the
 * workspace that orthdion_step asks for, so here the scratch lives in a fixed array that is part
 * of the library image itself: ORTHDION_NOALLOC_SCRATCH_BYTES bytes of device memory on every
 * GPU that loads the library, held until the process exits.
 *
 *  - X, M, G, Q: as for orthdion_step (device pointers, updated in place, G read only).
 *  - status_dev: optional DEVICE pointer to one int32; when not null the matrix's status flags
 *    (ORTHDION_STATUS_*) are copied there in stream order.  The factors P and R are not exposed.
 *  - A plan whose orthdion_workspace_bytes() exceeds ORTHDION_NOALLOC_SCRATCH_BYTES is rejected
 *    with ORTHDION_ERR_WORKSPACE (and a message on stderr); nothing is enqueued then.
 *  - The first call on a device looks up the device address of the array (no allocation).  Make
 *    that first call outside of any stream capture.
 *  - All calls share the one array, and it keeps whatever the previous call left in it; the step
 *    rewrites everything it later reads.  Two calls whose kernels overlap on the GPU (different
 *    streams, or several host threads) race on it: keep calls on one stream, or order them.
 *  - Results are those of orthdion_step on the same inputs.  Host-side bookkeeping may use the
 *    host heap; no CUDA allocation routine is called. */
#define ORTHDION_NOALLOC_SCRATCH_BYTES ((size_t)64 << 20)
int orthdion_step_noalloc(orthdion_t h, void* X, float* M, const void* G, float* Q,
                          int32_t* status_dev, void* stream);

/* Device pointers to the factors P (m x r) and R (n x r) that the last step left in the
 * workspace (for checks).  index = position in the grouped call, 0 for orthdion_step. */
int orthdion_get_factors(const orthdion_t* hs, int32_t count, int32_t index, void* workspace,
                         const float** P, const float** R);

/* Copies the `count` status words of the last step to host `flags` (synchronises `stream`). */
int orthdion_last_status(const orthdion_t* hs, int32_t count, void* workspace, void* stream,
                         int32_t* flags);

/* Optional per-step diagnostics (the paper's per-iteration quantities, appendix "Norms and Key
 * Quantities", and the effective-rank estimator of the adaptive-rank section), computed on the
 * device at the end of a step from what the step leaves behind.  mask: 0 off (default),
 * 1 factor diagnostics, 3 factor diagnostics and buffer norms (one more read of M and G).
 * Part of the plan's class: matrices with different masks are not batched together.
 * orthdion_last_diagnostics copies ORTHDION_DIAG_FLOATS floats per matrix to host `out`
 * (count * ORTHDION_DIAG_FLOATS floats; synchronises `stream`), in this order:
 *   [0] nu      = ||Q||_op (Proposition 3.1: 1 for ORTH, in [1, sqrt(r)] for COLNORM), the root of
 *                 the largest eigenvalue of Q^T Q by Lanczos iteration (at most 96 products with
 *                 Q^T Q; stops once the top Ritz value has settled to 1e-6)
 *   [1] erank   = exp(-sum_j p_j log p_j), p_j = ||R_j||_2 / sum_k ||R_k||_2
 *   [2] tr_t2   = <B, P Q^T> = <R, Q>  (Lemma 4.2; tr(T_2) for ORTH, sum of column norms for COLNORM)
 *   [3] norm_r  = ||R||_F = ||P^T B||_F
 *   [4] norm_m  = ||M'||_F   [5] norm_g = ||G||_F   (mask 3 only, else 0)
 *   [6] norm_b  = ||B||_F derived from ||M'||^2 = a^2 ||B||^2 - (2ab - b^2) ||R||^2, which holds
 *                 when P^T P = I (mask 3 only, else 0; 0 when a = 0)
 *   [7] number of products with Q^T Q the eigenvalue iteration used
 * A matrix whose step failed (ORTHDION_STATUS_RANK_DEFICIENT or _NONFINITE) reports NaN in every
 * slot; a matrix whose plan has diagnostics off reports zeros. */
#define ORTHDION_DIAG_FLOATS 8
int orthdion_set_diagnostics(orthdion_t h, int32_t mask);
int orthdion_last_diagnostics(const orthdion_t* hs, int32_t count, void* workspace, void* stream,
                              float* out);

/* Adaptive rank (appendix algorithm "Ada-Orth-Dion Rank Selection").  The estimate e_t is slot [1]
 * of the diagnostics (effective rank from the column norms of R).  Host arithmetic in double:
 *     ema    = alpha * e_t + (1 - alpha) * ema_prev
 *     target = ceil(gamma * ema)
 *     r_next = clip(target, r_min, r_max) rounded to the nearest multiple of `multiple` (tie: up)
 * r_min and r_max must be positive multiples of `multiple` (the paper rounds to 8; the TENSOR
 * engine needs 16), 0 <= alpha <= 1, gamma > 0 (the paper's text has 1.1, its table 1.425).  The
 * paper does not say how the average starts: pass ema_prev = e_t on the first step.  r_t is the
 * current rank (the rule is stated with it; the caller resizes when *r_next differs). */
int orthdion_rank_policy(double e_t, int32_t r_t, double ema_prev, int32_t r_min, int32_t r_max,
                         double alpha, double gamma, int32_t multiple, double* ema_out, int32_t* r_next);

/* The resize step of the rank-selection algorithm, for the one factor that is carried between
 * steps (the left factor is recomputed by every step): the warm-start factor is cut down or
 * extended to the new rank.  Q_new (n x r_new, device, row-major) receives the leading min(r_old, r_new) columns of
 * Q_old (n x r_old) and, when r_new > r_old, the columns of `pad` (n x (r_new - r_old), device,
 * row-major; may be null otherwise).  The paper does not say what the new columns hold: the caller
 * supplies them (any columns that keep B*Q of full column rank serve the power iteration, e.g.
 * N(0, 1/n) entries).  Q_new must not alias Q_old.  Enqueued on `stream`; the next step then uses
 * a plan created with r_new (plans of different rank are packed separately by the grouped step). */
int orthdion_resize_factor(const float* Q_old, int64_t n, int32_t r_old, float* Q_new, int32_t r_new,
                           const float* pad, void* stream);

/* Number of kernels this library has launched so far in this process (monotonic). */
int64_t orthdion_launch_count(void);

/* Optional per-stage timing.  Between profile_begin and profile_end every kernel launch of the
 * step functions is bracketed by a pair of CUDA events on the launching stream (at most
 * max_launches launches are recorded; profile_begin creates the events).  profile_end waits for
 * the recorded events and returns, per stage s < orthdion_stage_count(), the summed device time
 * ms[s] in milliseconds and the number of launches.  Stages are the kernels of the step: the
 * packers, Y = B*Q_prev, Gram, Cholesky+inverse, apply (the QR of the left-factor and normalisation steps),
 * R = B^T*P, ColNorm and the fused feedback/update pass.
 * Not thread-safe; meant for benchmarks. */
int orthdion_profile_begin(int32_t max_launches);
int orthdion_profile_end(int32_t n_stages, double* ms, int64_t* launches);
int32_t orthdion_stage_count(void);
const char* orthdion_stage_name(int32_t stage);

/* Library/kernels self-description: returns a static string naming the build (arch, engines). */
const char* orthdion_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ORTHDION_H_ */
