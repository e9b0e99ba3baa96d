/*
 * kurtail.h -- C ABI of libkurtail, a B200 (sm_100a) implementation of KurTail
 * rotation learning (arXiv 2503.01483): find an orthogonal R (d x d) that
 * minimises the kurtosis loss of the rotated calibration activations Y = X R.
 *
 * General conventions
 * -------------------
 * Pointers.  Every matrix pointer is a DEVICE pointer unless the parameter is
 *   documented "host".  Matrices are row-major.  The caller owns X, R, dR, the
 *   code/scale outputs and the workspace; the library never frees or
 *   reallocates them, and allocates no device memory after kt_create().
 * Shapes.  N = number of tokens (rows of X), any N >= 1 (ragged tails are
 *   handled).  d = channels, a multiple of 128.  X.ld >= d in elements; the
 *   base of X must be 16-byte aligned and X.ld * sizeof(element) a multiple of
 *   16 (the tiles are fetched by TMA).  R and dR are dense d x d float32,
 *   16-byte aligned.
 * Precision.  X is used as bfloat16 (float32 X is rounded once on entry), R is
 *   kept in float32 and enters the token GEMMs in a 16-bit form: float16
 *   against an exact float16 re-encoding of X's rows, or bfloat16 terms (see
 *   kt_config.forward_terms and forward_bf16); all products accumulate in
 *   float32 on the tensor cores.
 * Stream.  All work is issued on the stream given to kt_create().  Calls that
 *   return a host scalar synchronise that stream; the others are stream
 *   ordered and return after enqueueing.
 * Errors.  Every call returns a kt_status; nothing throws, aborts or prints.
 *   Argument errors are detected before any work is enqueued and leave all
 *   outputs untouched.  Device-side waits are bounded; if one runs out the
 *   kernel records it and the next synchronising call returns KT_ERR_TIMEOUT.
 *   There is no CPU or library fallback: a device that is not sm_100 gives
 *   KT_ERR_ARCH.
 */
#ifndef KURTAIL_H_
#define KURTAIL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kt_ctx kt_ctx;

typedef enum {
  KT_OK = 0,
  KT_ERR_INVALID_ARG = 1, /* null pointer, negative count, unknown enum     */
  KT_ERR_SHAPE = 2,       /* d not a multiple of 128, N < 1, ld < cols      */
  KT_ERR_ALIGN = 3,       /* base or leading dimension not 16-byte aligned  */
  KT_ERR_WORKSPACE = 4,   /* workspace missing or smaller than required     */
  KT_ERR_ARCH = 5,        /* current device is not compute capability 10.x  */
  KT_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed              */
  KT_ERR_NONFINITE = 7,   /* the loss came out NaN/Inf (outputs are written)*/
  KT_ERR_TIMEOUT = 8,     /* a bounded device-side wait ran out             */
  KT_ERR_TOO_LARGE = 9,   /* kt_kurtosis_loss_noalloc: N or d above its maximum */
  KT_ERR_COOPERATIVE = 10,/* the one-launch orthogonal step (d <= 512) needs 128
                             CTAs resident at once and the device cannot hold
                             them: set kt_config.small_d_orth = 0            */
  KT_ERR_REDUCE = 11      /* kt_fit_sharded: the caller's reduce hook failed   */
} kt_status;

/* Element types.  X is KT_BF16 or KT_F32; KT_F64 only names the type of a buffer
 * handed to a kt_reduce_fn. */
typedef enum { KT_BF16 = 0, KT_F32 = 1, KT_F64 = 2 } kt_dtype;

/* A row-major matrix: rows x cols elements of `dtype`, leading dimension `ld`
 * elements. */
typedef struct {
  const void* data;
  int32_t dtype; /* kt_dtype */
  int32_t reserved;
  int64_t rows, cols, ld;
} kt_mat;

/* Tunables.  kt_default_config() fills the defaults given in brackets. */
typedef struct {
  float kappa_target;   /* [1.8] kurtosis of the uniform distribution, the target
                           of the loss (Section 2, loss equation)              */
  int32_t cayley_iters; /* [2]   fixed-point iterations s of the Cayley step    */
  float q;              /* [0.5] contraction bound: alpha <= 2q / ||W||_F       */
  float eps;            /* [1e-8] added to ||W||_F in that bound                */
  float polish_thresh;  /* [1e-5] the Newton-Schulz polish runs when
                           max|R^T R - I| exceeds this; < 0: every step;
                           +inf: never.  (The guard measures R^T R from a
                           two-term bf16 split: its noise floor is about
                           2e-5/sqrt(d).)                                       */
  int32_t retract_terms;/* [0]   bf16 split terms of R in the product P0 = W R of
                           the retraction: 1..3 forces a count; 0 = chosen on
                           the device per step (one term while alpha*||W||_F *
                           2^-9 < 2.5e-6, else hi + lo), and series terms that
                           fall below float32 resolution are skipped (the
                           one-launch step for d <= 512, whose products are
                           float32, skips those terms by the same rule and
                           evaluates them all when a count is forced)          */
  int32_t guard_every;  /* [0]   kt_fit: k >= 1 measures R^T R - I every k-th step
                           (and after the last one); 0 = on the first and the
                           last step and in between whenever a device-side
                           bound on the accumulated drift reaches half of
                           polish_thresh; in this mode the polish already runs
                           at a quarter of polish_thresh, so that measurements
                           stay rare.  kt_orth_step always measures           */
  int32_t forward_terms;/* [0]   16-bit terms of R in the token GEMMs: 1 = R rounded
                           once (to float16, or to bf16 with forward_bf16);
                           2 = bf16 hi + lo (about 16 significant bits, twice
                           the MMA work); 0 = automatic: 2 when d <= 512 (with
                           few channels the rounding error of R is systematic
                           over tokens and one term can miss the 1e-3 loss
                           tolerance), else 1.  The single-pass d == 128 kernel
                           of kt_loss_grad / kt_fit uses one float16 term in
                           the automatic mode too and corrects the loss to
                           first order, L(R) = L(f16 R) + <dR, R - f16 R>, from
                           the gradient the same pass yields                    */
  int32_t small_d_fused;/* [1]   d == 128: kt_loss_grad / kt_fit use the single-pass
                           kernel (X read once per evaluation); 0 = the general
                           three-GEMM path                                      */
  int32_t small_d_orth; /* [1]   d <= 512: kt_orth_step runs as one cooperative
                           launch in float32 on the CUDA cores (128 CTAs; the
                           device must have at least 128 SMs free) instead of
                           about twenty tensor-core launches; 0 = general path  */
  int32_t optimizer;    /* [0]   kt_fit: 0 = Cayley SGD (kt_orth_step per step);
                           1 = Cayley Adam (kt_adam_step per step; the
                           workspace then also holds the d x d momentum)       */
  float beta1;          /* [0.9]  Cayley Adam: decay of the momentum M          */
  float beta2;          /* [0.99] Cayley Adam: decay of the scalar second moment */
  float adam_eps;       /* [1e-8] Cayley Adam: added under the square root      */
  int32_t norm_iters;   /* [2]   the per-step choices of retract_terms = 0 and
                           guard_every = 0 depend on the size of W as an
                           operator.  k >= 1: 2k products W v (a power
                           iteration from a fixed vector) estimate ||W||_2
                           from below; twice the estimate, capped by ||W||_F,
                           is used.  0: ||W||_F alone (a strict bound, but
                           loose by up to sqrt(d): more terms and more
                           measurements than needed).  alpha always uses
                           ||W||_F.  Ignored by the d <= 512 one-launch step   */
  int32_t backward_mode;/* [0]   where the backward pass takes Y from.  1 = a
                           second pass of the forward GEMM recomputes each Y
                           tile in tensor memory and nothing of Y is ever
                           written (2 N d^2 more flops).  0 = the forward pass
                           also stores Y as float16 (N*d*2 bytes of workspace;
                           every run of 128 entries of a row, 64 when d is not
                           a multiple of 256, carries its own power-of-two
                           factor, taken from the run's mean and sum of
                           squares, so the scale of X does not matter) and an
                           element-wise kernel reads it back: 4 bytes of
                           memory traffic per entry instead of 2 d flops, on a
                           B200 the cheaper side for d above a few hundred.
                           The loss and the row moments come from the float32
                           accumulators in every mode; the gradient of mode 0
                           differs from mode 1's by the rounding of Y to 11
                           significant bits (one or two parts in a thousand of
                           its norm).
                           2 = Y is stored as float32 (N*d*4 bytes): gradients
                           bit-identical to mode 1.  d == 128 with
                           small_d_fused needs none of this                    */
  int32_t cta_pairs;    /* [1]   1 = GEMMs with 256-wide column tiles run on
                           pairs of CTAs (thread-block clusters of two, one
                           MMA over both SMs' tensor cores, each CTA loading
                           half of the second operand); 0 = one CTA per tile  */
  int32_t loss_mode;    /* [0]   0 = one kurtosis per token (row) over its d
                           entries, loss = mean over tokens; 1 = the loss
                           equation of Section 2 taken literally: one kurtosis
                           over the concatenation of all N d entries of the
                           layer, loss = |kappa - kappa_target| (zero rows are
                           then part of the distribution; d == 128 uses the
                           general path)                                        */
  int32_t rmsnorm;      /* [0]   1 = the unit-gain RMSNorm of the small network of
                           Section 3, "Learning the Rotations", follows the
                           rotation: row t of X R is multiplied by
                           1 / sqrt(mean(x_t^2) + rms_eps) (an orthogonal R
                           keeps the norm of a row, so the factor is taken
                           from X, once per call; it is applied to the
                           float32 accumulator, X is neither copied nor
                           rounded again, and the gradient is the one with
                           respect to R of the normalised output with the
                           factor held fixed).  The per-token loss does not
                           depend on it; the whole-layer loss, kt_rotate and
                           the quantisation errors do                          */
  float rms_eps;        /* [1e-6] (0 is allowed: all-zero rows then get factor 0) */
  int32_t wait_limit_ms;/* [4000] bound of every device-side wait, in
                           milliseconds (<= 0: the default)                    */
  int32_t forward_bf16; /* [0]   operand type of the forward pass's token GEMMs
                           when R enters as one term (forward_terms == 1, or
                           automatic with d > 512).  0 = float16: the GEMMs
                           read a copy of X whose rows are scaled by a power
                           of two into float16's range (exact for bf16 data;
                           made once per call, N*d*2 bytes of workspace) and R
                           rounded to float16, and the epilogues undo the row
                           factor: 2^-12 instead of 2^-9 relative rounding of
                           R at the same tensor-core rate.  It matters once R
                           is no longer bf16-exact: with bf16 the loss and the
                           gradient are those at bf16(R), which after a few
                           steps from a Hadamard start is 2e-2 of the gradient's
                           norm away from the gradient at R (3e-3 with
                           float16).  1 = bf16 operands, X read in place       */
} kt_config;

/* Filled by kt_fit / kt_fit_layers (host memory). */
typedef struct {
  int32_t steps_done;
  int32_t degenerate_rows; /* rows skipped in the last evaluated loss          */
  double loss_first;       /* loss at R before the first step                   */
  double loss_last;        /* loss at R before the last step                    */
  double orth_err;         /* max|R^T R - I| seen by the last measuring step,
                              before its polish                                 */
  float alpha_last;        /* step size used by the last step                   */
  float w_norm_last;       /* ||W||_F of the last step                          */
  double* loss_history;    /* optional host array of `steps` entries, or NULL   */
  float w_op_last;         /* the size of W as an operator that the last step's
                              choices used (see kt_config.norm_iters)           */
  int32_t series_terms_last; /* series terms the last step evaluated            */
  int32_t p0_terms_last;   /* bf16 terms of R in the last step's product W R    */
  int32_t guards_run;      /* steps of this fit that measured R^T R - I         */
} kt_fit_report;

/* --- life cycle ---------------------------------------------------------- */

/* Fills *cfg with the defaults. */
void kt_default_config(kt_config* cfg);

/* Creates a context on the CURRENT device.  `cfg` may be NULL (defaults).
 * `cuda_stream` is a cudaStream_t (NULL = the legacy default stream).  Allocates
 * a few KiB of device and pinned host memory for scalars; released by
 * kt_destroy().  KT_ERR_ARCH on a device that is not sm_100. */
kt_status kt_create(kt_ctx** ctx, const kt_config* cfg, void* cuda_stream);
void kt_destroy(kt_ctx* ctx);
const char* kt_status_string(kt_status s);

/* Bytes of scratch the calls below need for an N x d problem whose X has
 * element type `x_dtype`.  Host-only; never touches the device. */
kt_status kt_workspace_bytes(const kt_ctx* ctx, int64_t N, int64_t d, int32_t x_dtype, size_t* bytes);

/* Hands the context a caller-allocated device buffer (256-byte aligned).  The
 * buffer must stay valid until replaced or the context is destroyed.  Calls
 * check that it is large enough for their N and d (KT_ERR_WORKSPACE if not). */
kt_status kt_set_workspace(kt_ctx* ctx, void* dev_ptr, size_t bytes);

/* --- rotation initialisers (Section 3: Hadamard rotations) ---------------- */

/* Writes R (d x d float32).  kind 0: identity.  kind 1: normalised Sylvester
 * Hadamard H[i][j] = (-1)^popcount(i & j) / sqrt(d); d must be a power of two
 * (KT_ERR_SHAPE otherwise).  Stream ordered. */
kt_status kt_init_rotation(kt_ctx* ctx, float* R, int64_t d, int32_t kind);

/* --- the loss (Section 2, Eq. 3 and the loss equation) -------------------- */

/* *loss (host) = (1/N) sum_t |kappa(Y_t) - kappa_target|, Y = X R, kappa the
 * ratio of the fourth central moment to the squared second central moment of
 * the d entries of row t.  Rows without spread (m2 <= 1e-6 * mean square) add
 * zero.  Y is never written to memory.  Synchronises. */
kt_status kt_kurtosis_loss(kt_ctx* ctx, kt_mat X, const float* R, double* loss);

/* Same loss, plus dR (d x d float32, device) = dL/dR = X^T (dL/dY), the
 * Euclidean gradient (Section 3, "Learning the Rotations": R is the weight of a
 * linear layer trained with this loss).  `loss` (host) may be NULL, in which
 * case the call is stream ordered and does not synchronise. */
kt_status kt_loss_grad(kt_ctx* ctx, kt_mat X, const float* R, float* dR, double* loss);

/* Test hook: per-row moments of Y = X R, moments[t] = {mean, m2, m3, m4}
 * (N x 4 float32, device).  Stream ordered. */
kt_status kt_row_moments(kt_ctx* ctx, kt_mat X, const float* R, float* moments);

/* Test hook: Y = X R as float32 (N x d dense, device).  Stream ordered. */
kt_status kt_rotate(kt_ctx* ctx, kt_mat X, const float* R, float* Y);

/* --- the step on the orthogonal group (Section 3, "Optimization in the
 *     Orthogonal Space": Cayley SGD) -------------------------------------- */

/* R <- retraction of R along -dR:  W = (dR R^T - R dR^T)/2,
 * alpha = min(lr, 2q/(||W||_F + eps)), Y0 = R - alpha W R,
 * Yi = R - alpha/2 W (R + Y(i-1)) for i = 1..cayley_iters, R <- Y(last), then
 * the orthogonality guard (see kt_config.polish_thresh).  The iteration is
 * evaluated as its Neumann series, which has the same partial sums:
 * Y_s = R - alpha sum_{k<=s} (-alpha/2)^k W^k (W R).  Built from d x d
 * tensor-core products only.  R is updated in place, one series term per
 * kernel; dR is read only.  Uses the workspace (sized for any N >= 1 and this
 * d).  Stream ordered.
 * d <= 512 with kt_config.small_d_orth (the default): the whole step is one
 * cooperative launch of 128 CTAs in float32 on the CUDA cores instead; all
 * 128 CTAs must be resident at once (a device with at least 128 free SMs),
 * else the call returns KT_ERR_COOPERATIVE and R is untouched. */
kt_status kt_orth_step(kt_ctx* ctx, float* R, const float* dR, int64_t d, float lr);

/* Cayley Adam (Section 3, "Optimization in the Orthogonal Space", names it as
 * the optimiser of the paper's runs and defers to the publication it cites;
 * the update below is that publication's algorithm for a square orthogonal
 * R).  With k = st->step + 1:
 *   M <- beta1 M + (1 - beta1) dR;   v <- beta2 v + (1 - beta2) ||dR||_F^2;
 *   r = (1 - beta1^k) sqrt(v / (1 - beta2^k) + adam_eps);
 *   W = (M R^T - R M^T) / (2 r);     M <- r W R   (momentum back on the tangent space);
 *   alpha = min(lr, 2q/(||W||_F + eps)); then the same fixed-point iteration
 *   and guard as kt_orth_step, started from Y0 = R - alpha W R.
 * R (device, d x d) and M (device, d x d float32, caller-owned, zero before
 * the first step) are updated in place; dR is read only.  *st (host) carries
 * v and the step count between calls: zero it before the first step; it is
 * read on entry and written on return.  beta1, beta2, adam_eps come from the
 * context's configuration.  d <= 512 takes the one-launch float32 step like
 * kt_orth_step (kt_config.small_d_orth), larger d the tensor-core path.  Uses
 * the workspace (sized for any N >= 1 and this d).  Synchronises. */
typedef struct {
  double v;        /* running mean of ||dR||_F^2 */
  int32_t step;    /* steps taken so far */
  int32_t reserved;
} kt_adam_state;
kt_status kt_adam_step(kt_ctx* ctx, float* R, const float* dR, float* M, kt_adam_state* st, int64_t d, float lr);

/* *err (host) = max|R^T R - I|.  Uses the workspace.  Synchronises. */
kt_status kt_orth_error(kt_ctx* ctx, const float* R, int64_t d, double* err);

/* `steps` x (kt_loss_grad; kt_orth_step) -- or kt_adam_step from a zero state
 * when kt_config.optimizer == 1 -- on the context's stream with no host
 * synchronisation in between; bit-identical to composing those calls when
 * guard_every == 1 (with the default 0 the two differ only in which steps
 * measure orthogonality).  R in/out.  `report` (host) may be NULL.  Synchronises at
 * the end.  On an argument error R is untouched; after a CUDA failure in the
 * middle of a step R may hold a partially applied step. */
kt_status kt_fit(kt_ctx* ctx, kt_mat X, float* R, int32_t steps, float lr, kt_fit_report* report);

/* kt_fit for one shard of the rows of a batch that is spread over several
 * processes or GPUs (one rotation over many tokens: Section 3, "Learning the
 * Rotations").  X_local holds this shard's rows; rows_total is the number of
 * rows of all shards together (the loss is the mean over all of them).  Every
 * step the library calls `reduce` from the host thread, while it enqueues the
 * step, for each device buffer that has to be summed over the shards:
 *   per-token loss:   the loss (1 x KT_F64), then dR (d*d x KT_F32);
 *   whole-layer loss: the batch mean (1 x KT_F64), its three central sums
 *                     (3 x KT_F64), then dR.
 * The hook must enqueue an in-place sum all-reduce of `count` elements of type
 * `dtype` (a kt_dtype) at dev_ptr on `cuda_stream` (the context's stream) --
 * e.g. ncclAllReduce -- and return 0; it must not synchronise the stream.  A
 * non-zero return ends the fit with KT_ERR_REDUCE.  Every shard then holds the
 * same gradient and takes the same orthogonal step, so the replicas of R stay
 * bit-identical without being exchanged, and nothing synchronises with the
 * host inside the loop.  reduce == NULL stands for a single shard; with
 * rows_total == X_local.rows the call is then kt_fit, bit for bit.  The
 * report's degenerate_rows counts this shard's rows only. */
typedef int32_t (*kt_reduce_fn)(void* user, void* dev_ptr, int64_t count, int32_t dtype, void* cuda_stream);
kt_status kt_fit_sharded(kt_ctx* ctx, kt_mat X_local, float* R, int64_t rows_total, kt_reduce_fn reduce, void* user,
                         int32_t steps, float lr, kt_fit_report* report);

/* Layer-wise driver (Section 3, "Training Cost": activations are stored per
 * layer, then one rotation is optimised at a time).  X_layers[l] and
 * R_layers[l] for l in [first_layer, L) are fitted one after another on the
 * stream; all layer buffers stay resident in device memory.  All layers must
 * share N, d and dtype.  per_layer (host, L entries) may be NULL. */
kt_status kt_fit_layers(kt_ctx* ctx, const kt_mat* X_layers, float* const* R_layers, int32_t L,
                        int32_t first_layer, int32_t steps, float lr, kt_fit_report* per_layer);

/* One rotation shared by several activation buffers (Section 3, "Learning the
 * Rotations": the stored inputs of all transformer layers and of both blocks
 * are shuffled and a single R1 is trained on them).  X_bufs[0..n_bufs) are
 * device matrices of equal rows, cols, ld and dtype (n_bufs <= 4096); a
 * "sample" is a run of rows_per_sample consecutive rows (rows must be a
 * multiple of it), numbered id = buffer * (rows / rows_per_sample) + index
 * within the buffer.  Step k fits on the minibatch of the `batch` samples
 * order[k*batch .. (k+1)*batch): their rows, in that order, form a matrix of
 * batch*rows_per_sample rows (gathered in the workspace into the operand
 * forms of the token GEMMs; never more than one minibatch at a time), and the
 * step is the one kt_fit takes on that matrix, bit for bit (loss_mode,
 * rmsnorm, optimizer as configured).  The shuffle is the caller's: `order` (host, steps*batch
 * entries) is an input, so that a run can be reproduced exactly.  Needs a
 * workspace of kt_fit_shared_workspace_bytes().  KT_ERR_INVALID_ARG if an id
 * is out of range (checked before any work).  Synchronises at the end. */
kt_status kt_fit_shared_workspace_bytes(const kt_ctx* ctx, int64_t rows_per_sample, int32_t batch, int64_t d,
                                        size_t* bytes);
kt_status kt_fit_shared(kt_ctx* ctx, const kt_mat* X_bufs, int32_t n_bufs, int64_t rows_per_sample,
                        const int32_t* order, int32_t batch, float* R, int32_t steps, float lr,
                        kt_fit_report* report);

/* kt_fit_shared for one shard of every minibatch: this process gathers `batch`
 * samples per step from its own buffers (its own `order`), the other shards
 * theirs; rows_total = rows of a whole minibatch over all shards.  `reduce` as
 * in kt_fit_sharded. */
kt_status kt_fit_shared_sharded(kt_ctx* ctx, const kt_mat* X_bufs, int32_t n_bufs, int64_t rows_per_sample,
                                const int32_t* order, int32_t batch, float* R, int64_t rows_total,
                                kt_reduce_fn reduce, void* user, int32_t steps, float lr, kt_fit_report* report);

/* kt_fit with HOST buffers: copies X_host (N x d, pinned or pageable host
 * memory) into X_dev_staging (device, N*ld elements), R_host (d x d float32)
 * into R_dev, fits, and copies R back to R_host.  The copies run on the
 * context's stream. */
kt_status kt_fit_host(kt_ctx* ctx, kt_mat X_host, void* X_dev_staging, float* R_host, float* R_dev,
                      int32_t steps, float lr, kt_fit_report* report);

/* --- 4-bit fake quantisation (Section 2, "Uniform Quantization for k-bit
 *     Precision", symmetric case with k = 4, and Eq. 1) -------------------- */

/* *mse (host) = mean over all N*d entries of (Y - Q(Y))^2 with Y = X R and, per
 * token, s = max|Y_t| / 7, Q(y) = clamp(round_half_even(y / s), -7, 7) * s.
 * Y is recomputed instead of stored.  Synchronises. */
kt_status kt_quant4_error(kt_ctx* ctx, kt_mat X, const float* R, double* mse);

/* The general quantizer of the same paragraph, per token (one step and one
 * shift per row), k = bits in 2..8:
 *   symmetric:   b = 0,               s = clip * max|y| / (2^(k-1) - 1),
 *                codes in [-(2^(k-1) - 1), 2^(k-1) - 1];
 *   asymmetric:  b = clip * min(y),   s = (clip * max(y) - b) / (2^k - 1),
 *                codes in [0, 2^k - 1]   (Section 4, "Setup": used for the
 *                KV cache);
 *   Q(y) = clamp(round_half_even((y - b) / s), lo, hi) * s + b;  s == 0 -> Q(y) = b.
 * `clip` in (0, 1] shrinks the range towards zero before the step is formed
 * ("Setup" clips activations; 1 = no clipping, the definition of Section 2).
 * "Setup" words the clipping of activations as "a quantile of 0.98", which can
 * be read two ways; both are here.  clip_mode 0: `clip` is a ratio, as above.
 * clip_mode 1 (symmetric only): `clip` is a quantile level and the range is the
 * clip-quantile of the row's |y| -- with the d magnitudes sorted,
 * a[0] <= ... <= a[d-1], and h = clip (d - 1) = k + t (k integer, 0 <= t < 1),
 * range = a[k] + t (a[k+1] - a[k]); entries beyond it saturate.  The order
 * statistic is exact (a selection on the float32 bit patterns), the
 * interpolation is float32.  A quantile needs a whole row of Y at once, so
 * this mode works on a given Y (kt_quant_codes, kt_quant_error_given), not
 * inside the GEMM passes of kt_quant_error (KT_ERR_INVALID_ARG there).
 * All decisions in IEEE float32.  {4, 0, 1.0, 0} is kt_quant4_error. */
typedef struct {
  int32_t bits;       /* 2..8 */
  int32_t asymmetric; /* 0 or 1 */
  float clip;         /* (0, 1] */
  int32_t clip_mode;  /* 0 = ratio of the row's range, 1 = quantile level of |y| */
} kt_quant_spec;

/* *mse (host) = mean over all N*d entries of (Y - Q(Y))^2, Y = X R recomputed in
 * two GEMM passes (row range, then error).  KT_ERR_INVALID_ARG for a spec out
 * of range.  Synchronises. */
kt_status kt_quant_error(kt_ctx* ctx, kt_mat X, const float* R, const kt_quant_spec* spec, double* mse);

/* Test hook: quantise a given float32 Y (N x d dense, device) with `spec`:
 * codes (N x d int16), scales s and shifts b (N float32 each), all device.
 * No workspace needed.  Stream ordered. */
kt_status kt_quant_codes(kt_ctx* ctx, const float* Y, int64_t N, int64_t d, const kt_quant_spec* spec,
                         int16_t* codes, float* scales, float* shifts);

/* *mse (host) = mean over all N*d entries of (Y - Q(Y))^2 for a given float32 Y
 * (N x d dense, device; e.g. from kt_rotate), any `spec` including clip_mode 1
 * (Section 2, Eq. 1 with the quantizer of "Setup").  One block per row, then a
 * fixed-order sum; uses the first N*8 bytes of the workspace
 * (KT_ERR_WORKSPACE if it is smaller).  Synchronises. */
kt_status kt_quant_error_given(kt_ctx* ctx, const float* Y, int64_t N, int64_t d, const kt_quant_spec* spec,
                               double* mse);

/* Success rate of Section 3 (the comparison of per-token maxima): *rate (host) =
 * the fraction of tokens t with max_j |(X R_a)_tj| < max_j |(X R_b)_tj|.  R_b may
 * be NULL: the un-rotated token itself (max_j |X_tj|).  Uses the workspace.
 * Synchronises. */
kt_status kt_rowmax_success(kt_ctx* ctx, kt_mat X, const float* R_a, const float* R_b, double* rate);

/* Test hook: quantise a given float32 Y (N x d dense, device): codes (N x d
 * int8, device) and scales (N float32, device).  Float32 IEEE divide and
 * round-half-even decide the codes.  No workspace needed.  Stream ordered. */
kt_status kt_quant4_codes(kt_ctx* ctx, const float* Y, int64_t N, int64_t d, int8_t* codes, float* scales);

/* --- a loss call that allocates nothing ----------------------------------- */

/* (The paper has no counterpart to this call; it exists for deployment.)
 *
 * kt_kurtosis_loss for callers that cannot allocate device memory: code running
 * inside a memory pool that owns the whole GPU, a plug-in that is forbidden to
 * call cudaMalloc because the host application budgets every byte, or a
 * real-time loop where an allocation (an implicit device synchronisation) is not
 * acceptable.  It needs no kt_ctx and no workspace: its scratch -- the bf16
 * copies of R^T, the per-tile and per-row moment records, the block sums and the
 * status words -- is a fixed 8 MiB array compiled into the library, which every
 * GPU that loads the library holds until the process exits.  Neither this call
 * nor anything it uses calls cudaMalloc, cudaFree or an allocating routine.
 *
 *   X        bf16 only, device, N <= KT_NOALLOC_MAX_N rows, d <= KT_NOALLOC_MAX_D
 *            (same alignment rules as elsewhere); larger problems return
 *            KT_ERR_TOO_LARGE and float32 X returns KT_ERR_INVALID_ARG, with
 *            nothing enqueued.
 *   R        d x d float32, device.
 *   loss_dev DEVICE pointer to one double (8-byte aligned) that receives the
 *            loss.  The call is stream ordered on `cuda_stream` and does not
 *            synchronise; read the value after synchronising that stream.
 *            Since the call never reads anything back, it cannot return
 *            KT_ERR_TIMEOUT or KT_ERR_NONFINITE: if one of its kernels gave up
 *            a bounded wait, *loss_dev is NaN, and a non-finite loss is simply
 *            stored.  Treat a NaN there as a failed call.
 *   X, R and loss_dev must be device (or managed) memory of the CURRENT
 *   device, whose copy of the array is the one used; KT_ERR_INVALID_ARG
 *   otherwise.
 *
 * The first call on each device looks up the device address of the built-in
 * array and a driver entry point, with that device current.  Make that first
 * call before starting any stream capture.
 * All calls on a device share the one array, which keeps the previous call's
 * contents (the call clears the words that must start at zero itself).  Two
 * calls that overlap on the GPU -- different streams, or different host threads
 * without ordering between their streams -- race on it; order them yourself.
 * The default configuration (kappa_target 1.8, forward_terms auto) applies,
 * with bf16 operands throughout (forward_bf16 = 1: the float16 copy of X that
 * the regular entry points make would not fit the built-in array). */
#define KT_NOALLOC_MAX_N 16384
#define KT_NOALLOC_MAX_D 1024
kt_status kt_kurtosis_loss_noalloc(kt_mat X, const float* R, double* loss_dev, void* cuda_stream);

/* --- error-path test hook ------------------------------------------------- */

/* Enqueues a one-warp kernel that waits, through the same bounded wait every
 * kernel of this library uses, on a barrier that nothing ever signals, with a
 * limit of limit_ms (1..1000) milliseconds.  The wait runs out, the kernel
 * returns normally and records it: the next synchronising call on this context
 * returns KT_ERR_TIMEOUT (and clears the record); the call after that works
 * again.  Nothing traps or faults.  Stream ordered. */
kt_status kt_test_wait_timeout(kt_ctx* ctx, int32_t limit_ms);

/* --- measurement ---------------------------------------------------------- */

/* Device time of the tensor-core GEMM launches, by role, between
 * kt_profile_begin() and kt_profile_end(): 0 forward (Y = X R with the moment
 * epilogue; Section 2, Eq. 3), 1 backward-A (recompute Y, write dL/dY),
 * 2 backward-B (dR = X^T dL/dY), 3 the d x d products of the Cayley step and its
 * guard (Section 3), 4 the two quantizer passes (Section 2, Eq. 1), 5 the
 * single-pass loss+gradient kernel used when d == 128.  Times come
 * from CUDA events recorded on the context's stream around each launch (up to
 * 8192 launches per window).  launches_total counts every kernel this library
 * launched in the window.  kt_profile_end() synchronises; `out` is host memory. */
typedef struct {
  int64_t launches_total;
  int32_t gemm_launches[8];
  float gemm_ms[8];
} kt_profile;
kt_status kt_profile_begin(kt_ctx* ctx);
kt_status kt_profile_end(kt_ctx* ctx, kt_profile* out);

#ifdef __cplusplus
}
#endif
#endif /* KURTAIL_H_ */
