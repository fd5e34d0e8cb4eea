/*
 * dartquant.h -- C ABI of the B200 (sm_100a) rotational-distribution-calibration
 * library.
 *
 * One calibration iteration is the loop body of Algorithm 1 of the DartQuant
 * paper: R <- Q factor of qr(Z) (QR-Orth, Sec. 4.3 / Algorithm 2), O <- X R,
 * L <- Whip(O) (Eq. 4), Z <- Z - eta dL/dZ.  Every step runs in CUDA kernels of
 * this library; there is no CPU fallback.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.
 *   - Matrices are row-major.  X is [batch][n_tokens][ldx] (one token per row),
 *     latents / rotations are [batch][d][d] fp32.
 *   - One process may use the library on several devices (a handle belongs to the device that was
 *     current at dq_calib_init; per-device kernel attributes are set on first use of each device).
 *   - Every call returns a dq_status; nothing throws, aborts or traps.  Device
 *     side problems (rank-deficient latent, non-finite loss, a wait that ran
 *     out) are recorded in a device status word read by dq_calib_status().  The
 *     first error wins and stays until dq_calib_set_latent or one of the
 *     dq_calib_set_* configuration calls clears it; while it is set, the kernels
 *     that update the latent (or the Cayley iterate) and the optimiser state
 *     change nothing, so the parameter stays at the last good iterate.
 *   - All work is enqueued on the stream given at init; calls are asynchronous
 *     with respect to the host unless stated otherwise.
 *   - Notation: R is always the rotation (the orthogonal factor of Z = R U),
 *     U the upper-triangular factor with positive diagonal.
 */
#ifndef DARTQUANT_H_
#define DARTQUANT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dq_calib dq_calib_t; /* opaque, owned by the library */

typedef enum {
  DQ_OK = 0,
  DQ_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad enum          */
  DQ_ERR_UNSUPPORTED = 2, /* shape / dtype / path combination not implemented   */
  DQ_ERR_ALLOC = 3,       /* device allocation failed                           */
  DQ_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed                  */
  DQ_ERR_SINGULAR = 5,    /* latent is (numerically) rank deficient: U^-T undefined */
  DQ_ERR_NONFINITE = 6,   /* loss became NaN/Inf                                */
  DQ_ERR_TIMEOUT = 7,     /* a bounded in-kernel wait gave up                   */
  DQ_ERR_NOT_CONVERGED = 8 /* DQ_QR_ITERATIVE: one step moved the latent too far     */
} dq_status;

enum { DQ_FP32 = 0, DQ_BF16 = 1 };             /* x_dtype                       */
enum { DQ_PATH_FP32 = 0, DQ_PATH_BF16_TC = 1 }; /* arithmetic of the X R / X^T G contractions */
enum { DQ_MEAN_TOKENS = 0, DQ_SUM_TOKENS = 1 }; /* reduction of Eq. 4 over token rows */
enum { DQ_SGD = 0, DQ_SGD_MOMENTUM = 1, DQ_ADAM = 2 }; /* optimiser (Algorithm 1, update step; Sec. 4.3: "SGD or Adam") */

typedef struct {
  int32_t d;         /* channels = size of the rotation; multiple of 64 (fp32 path) or 128 (tensor-core path); <= 8192 */
  int64_t n_tokens;  /* tokens per problem; any positive count (fp32 path) or a multiple of 256 (tensor-core path) */
  int32_t batch;     /* independent problems (e.g. attention heads); >= 1       */
  int32_t x_dtype;   /* DQ_FP32 | DQ_BF16                                       */
  int32_t path;      /* DQ_PATH_FP32: fp32 FMA contractions (needs DQ_FP32 X);
                        DQ_PATH_BF16_TC: bf16 tensor-core contractions with fp32 accumulation (needs DQ_BF16 X) */
  int32_t reduction; /* DQ_MEAN_TOKENS (default reading of Algorithm 1's loss step) | DQ_SUM_TOKENS */
  int32_t optimizer; /* DQ_SGD here; others via dq_calib_set_optimizer          */
  float lr;          /* eta                                                     */
  int64_t ldx;       /* row stride of X in elements (>= d; a multiple of 8 on the tensor-core path); problems are n_tokens*ldx apart */
} dq_calib_config;

/* Algorithm 1, hand-off before the loop: bind calibration activations and the initial
 * latent.  d_X is BORROWED (must outlive the handle; only dq_calib_run_epochs writes it).  d_Z0
 * ([batch][d][d] fp32) is COPIED.  cuda_stream is a cudaStream_t (NULL = legacy
 * default stream).  Allocates every workspace the step needs.
 * Errors: INVALID_ARG, UNSUPPORTED, ALLOC, CUDA.  *out is NULL on error. */
dq_status dq_calib_init(dq_calib_t** out, const dq_calib_config* cfg, const void* d_X,
                        const float* d_Z0, void* cuda_stream);

/* Algorithm 1's loop, exactly n_steps iterations.  d_loss_out (nullable) is a
 * device array [n_steps][batch] fp32; entry k is L(Z_k), the loss BEFORE the
 * k-th update.  No host synchronisation. */
dq_status dq_calib_step(dq_calib_t* h, int32_t n_steps, float* d_loss_out);

/* Sec. 4.3: the rotation of the CURRENT latent, i.e. the orthogonal factor of
 * Z = R U with diag(U) > 0 (recomputed if the latent changed since the last
 * factorisation).  d_R_out is caller-owned [batch][d][d] fp32. */
dq_status dq_calib_get_rotation(dq_calib_t* h, float* d_R_out);

/* Sec. 3 (Y = X R): apply a rotation to activations and materialise the result.
 * x_dtype selects both the storage type of X / Y and the arithmetic (DQ_FP32:
 * fp32 FMA; DQ_BF16: bf16 tensor cores, fp32 accumulation, bf16 output).
 * X is [n][ldx], Y is [n][ldy], R is [d][d] fp32, all device, no aliasing. */
dq_status dq_rotate_apply(const void* d_X, int32_t x_dtype, int64_t n, int32_t d, int64_t ldx,
                          const float* d_R, void* d_Y, int64_t ldy, void* cuda_stream);

/* (No counterpart in the paper: a packaging variant of dq_rotate_apply for bf16 activations.)
 * The same Y = X R, for callers that must not allocate device memory: a serving process that
 * handed all of HBM to its own arena at start-up (a later cudaMalloc would fail or fragment
 * it), or a latency-critical loop where the implicit device synchronisation of cudaFree is
 * not acceptable.  dq_rotate_apply allocates and frees a bf16 copy of R^T on every call; this
 * variant keeps that copy in a fixed device array inside the library (8 MiB, held by every GPU
 * that loads the library until the process exits) and calls no cudaMalloc / cudaFree or any
 * other allocating routine.
 *   - X, Y: bf16 [n][ldx] / [n][ldy]; R: fp32 [d][d]; all device, caller-owned, no aliasing.
 *   - d <= 2048 (the size of the fixed array), d % 128 == 0, n % 128 == 0, ldx % 8 == ldy % 8 == 0;
 *     anything else returns DQ_ERR_UNSUPPORTED and launches nothing.
 *   - The first call on each device also looks up the array's device address; make that call
 *     once, with that device current, before any stream capture.  It is also the call on which the
 *     CUDA runtime may load this library's kernels (and the array itself) onto the device, which
 *     takes device memory once: make it before the caller's arena takes the rest of HBM.
 *   - All calls share the one array.  Each call rewrites the part it uses before reading it, so
 *     calls on one stream are independent; calls that overlap on the GPU (different streams or
 *     threads without ordering between them) race on it and must be serialised by the caller. */
dq_status dq_rotate_apply_static(const void* d_X, int64_t n, int32_t d, int64_t ldx, const float* d_R,
                                 void* d_Y, int64_t ldy, void* cuda_stream);

/* What the paper measures a rotation by (Sec. 4.1, Eq. 1; appendix on outliers and quantisation
 * errors), for O = X R with X [n][ldx] (DQ_FP32 or DQ_BF16) and R fp32 [d][d], all device:
 *   d_out[0] = number of entries with |o| > tau                                  (Eq. 1 over all tokens)
 *   d_out[1] = mean squared error of per-token asymmetric uniform quantisation of O to `bits` bits:
 *              scale = (max - min) / (2^bits - 1), zero = round(-min / scale),
 *              q = clamp(round(o / scale) + zero, 0, 2^bits - 1), dequantised = scale (q - zero)
 * d_out is a device double[2], written on the stream.  O is computed with bf16 tensor cores for
 * DQ_BF16 (d % 128 == 0, n % 128 == 0) and fp32 FMA for DQ_FP32.  Allocates stream-ordered scratch.
 * Errors: INVALID_ARG (null, bits outside 1..16, tau < 0), UNSUPPORTED, ALLOC, CUDA. */
dq_status dq_eval_rotation(const void* d_X, int32_t x_dtype, int64_t n, int32_t d, int64_t ldx, const float* d_R,
                           float tau, int32_t bits, double* d_out, void* cuda_stream);

/* Algorithm 1, X <- token_sampling(X), and the mini-batches of the hyper-parameter appendix:
 * d_out[i] = d_X[pi(first + i)] for 0 <= i < count, where pi is a pseudo-random permutation of the
 * token rows [0, n_total) fixed by `seed` (uniform sampling without replacement: a Feistel network
 * with cycle walking over the Philox4x32-10 generator).  A sample of k tokens is first = 0,
 * count = k; mini-batches are consecutive windows; use another seed for another epoch.
 * X is [n_total][ldx], out is [count][ldo], both device, x_dtype DQ_FP32 or DQ_BF16, rows and row
 * strides multiples of 16 bytes (else DQ_ERR_UNSUPPORTED).  To calibrate on the batch, gather into
 * the buffer bound at dq_calib_init and call dq_calib_refresh_inputs. */
dq_status dq_gather_tokens(const void* d_X, int32_t x_dtype, int64_t n_total, int32_t d, int64_t ldx, uint64_t seed,
                           int64_t first, int64_t count, void* d_out, int64_t ldo, void* cuda_stream);

/* Mini-batch use (the paper feeds the loop with batches of sampled tokens): the
 * caller overwrote the borrowed activation buffer d_X in place (same shape) on
 * the handle's stream.  Every kernel reads the activations in place (no copy of them is
 * derived or kept), so today this call only orders the handle's internal stream after the
 * caller's writes; call it all the same after rewriting d_X. */
dq_status dq_calib_refresh_inputs(dq_calib_t* h);

/* Optimiser of the latent (Sec. 4.3: QR-Orth works with any standard optimiser; the paper reports
 * SGD and Adam).  Resets the optimiser state (moments, step count) and replaces the learning rate.
 *   DQ_SGD:          Z <- Z - lr g                                   (beta1, beta2, eps ignored)
 *   DQ_SGD_MOMENTUM: v <- beta1 v + g;  Z <- Z - lr v                 (beta1 = momentum)
 *   DQ_ADAM:         m <- beta1 m + (1 - beta1) g;  v <- beta2 v + (1 - beta2) g^2;
 *                    Z <- Z - lr (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
 * Errors: INVALID_ARG (bad enum, betas outside [0, 1), eps < 0), ALLOC, CUDA. */
dq_status dq_calib_set_optimizer(dq_calib_t* h, int32_t optimizer, float lr, float beta1, float beta2, float eps);

/* How the QR-Orth forward (Sec. 4.3: Z = R U) is computed on the tensor-core path.  Both
 * give the same unique factors (diag(U) > 0).
 *   DQ_QR_ITERATIVE (default): incremental.  Blocked Householder QR (Algorithm 2 in compact-WY
 *     form) only when no factors of a nearby latent are known (first step, after
 *     dq_calib_set_latent or a change of method).  Afterwards, with the previous step's W_old = U_old^-1,
 *     Zh = Z W_old is close to orthogonal whatever Z is, its upper factor I + T is the fixed point
 *     of T <- striu(E - T^T T) + diag(E - T^T T) / 2 with E = Zh^T Zh - I, reached by sweeps of
 *     triangular tensor-core GEMMs (no dependent column steps) that start from the previous step's
 *     T^T T, and R = Zh (I + T)^-1, W = W_old (I + T)^-1 (the inverse of I + T from a few more triangular
 *     products; U itself is not formed).  The sweeps stop by themselves: each is skipped (by a
 *     device-side flag, so the launch sequence and a captured graph stay fixed) once the sweep before it
 *     moved no entry by more than 1e-5; the first two use a plain bf16 product, later ones and, after
 *     a step large enough to need them, the first-order correction products use split-bf16 operands.
 *     At most n_iters + 3 sweeps.  If the last of those still moved an entry, one optimiser step has
 *     moved the latent too far: the status word becomes DQ_ERR_NOT_CONVERGED and, as after every
 *     device-side error, the update kernels leave the latent and the optimiser state untouched from
 *     then on: the latent stays at the last good iterate.  Recover with
 *     dq_calib_set_qr_method(h, DQ_QR_HOUSEHOLDER, 0), more sweeps or a lower learning rate, and step
 *     again.  n_iters <= 0 selects the default (5 on this route: the paper's SGD steps need one
 *     sweep; an optimiser that moves every entry by its learning rate, such as Adam, may need more);
 *     at most 64.
 *   DQ_QR_HOUSEHOLDER: blocked Householder QR at every step; no assumption on the step size.
 * The call clears the status word.  For d == 128 (any path) the same two methods exist as kernels that
 * keep a whole latent in shared memory; there the sweeps stop as soon as no entry moves (one more is
 * taken) and n_iters only bounds them (4 n_iters).  On the fp32 path with d <= 1024 the incremental
 * factorisation runs on fp32 FMA products (up to n_iters + 3 sweeps, switched off the same way); larger fp32
 * latents are always factored with Householder. */
enum { DQ_QR_HOUSEHOLDER = 0, DQ_QR_ITERATIVE = 1 };
dq_status dq_calib_set_qr_method(dq_calib_t* h, int32_t method, int32_t n_iters);

/* Algorithm 1's loop around the step: token sampling and mini-batches (hyper-parameter appendix: a
 * fraction of the captured tokens per epoch, fixed batch size, several epochs).
 * d_pool: device, [n_pool][ld_pool] token rows of the handle's x_dtype, borrowed, never written.
 * Epoch e draws the seeded permutation pi of dq_gather_tokens with seed + e and uses its first
 * floor(sample_ratio * n_pool) rows (sampling without replacement), cut into optimiser steps of
 * accum micro-batches of the handle's n_tokens rows each; an incomplete last step is dropped.
 * Every micro-batch is gathered into the activation buffer given to dq_calib_init, WHICH THIS CALL
 * OVERWRITES (it must be writable device memory of n_tokens rows); dL/dR and the loss of a step are
 * the mean over all accum * n_tokens tokens of the step (gradient accumulation: the sum with
 * DQ_SUM_TOKENS), then one QR backward / optimiser update follows.  The paper does not say how tokens
 * are drawn or batched; this is the reading.  d_loss_out: nullable, device
 * [n_epochs * steps_per_epoch] with steps_per_epoch = floor(floor(sample_ratio * n_pool) /
 * (accum * n_tokens)); the product runs in double precision on the float sample_ratio.
 * h_steps_out: nullable HOST pointer, receives the number of optimiser steps enqueued.
 * Asynchronous like dq_calib_step; steps are not replayed from a graph (the gather changes).
 * Errors: INVALID_ARG (null, sizes, ratio outside (0, 1], no complete step), UNSUPPORTED (batch > 1),
 * CUDA. */
dq_status dq_calib_run_epochs(dq_calib_t* h, const void* d_pool, int64_t n_pool, int64_t ld_pool,
                              float sample_ratio, int32_t accum, int32_t n_epochs, uint64_t seed,
                              float* d_loss_out, int64_t* h_steps_out);

/* Arithmetic of the QR-Orth backward (Sec. 4.3: dL/dZ from dL/dR, Z = R U) on the tensor-core path for
 * d >= 256.  dL/dR carries the bf16 rounding of the rotation operand and of dL/dO (a few percent), so by
 * default (split = 0) its d x d products run on plain bf16 operands with fp32 accumulation (2^-9 relative);
 * split != 0 runs them on split-bf16 operands (three MMAs per product, about 2^-17).  No effect elsewhere. */
dq_status dq_calib_set_backward_precision(dq_calib_t* h, int32_t split);

/* The calibration objective.  DQ_OBJ_WHIP (default) is Eq. 4.  The other three are the objectives the
 * ablation of Sec. 5.3 compares it with; the paper names them without formulas, so they are read as
 * per-token statistics over the d channels of the rotated token o = x R (as Eq. 4 is per token),
 * averaged over tokens like the Whip loss (or summed, with DQ_SUM_TOKENS):
 *   DQ_OBJ_VARIANCE: (1/d) sum_j (o_j - mean(o))^2
 *   DQ_OBJ_KURTOSIS: m4 / m2^2 - 3 with m_p = (1/d) sum_j (o_j - mean(o))^p   (excess kurtosis)
 *   DQ_OBJ_QUANT:    (1/d) sum_j (o_j - Q(o)_j)^2, Q = per-token asymmetric uniform quantiser to `bits`
 *                    bits (the one of dq_eval_rotation); derivative with the grid held fixed and rounding
 *                    piecewise constant: (2/d) (o_j - Q(o)_j)
 * These need statistics of the whole token before any entry of dL/dO, so the rotated activations are
 * materialised chunk by chunk in fp32 instead of staying in tensor memory; everything after dL/dO
 * (contraction with X, QR backward or Cayley update, optimiser) is unchanged.  bits: 1..16, <= 0 selects
 * 4; ignored unless DQ_OBJ_QUANT.  A token whose rotated entries are all equal makes the kurtosis
 * undefined: the loss becomes non-finite and the status word DQ_ERR_NONFINITE.
 * Errors: INVALID_ARG (bad enum, bits > 16), ALLOC, CUDA. */
enum { DQ_OBJ_WHIP = 0, DQ_OBJ_VARIANCE = 1, DQ_OBJ_KURTOSIS = 2, DQ_OBJ_QUANT = 3 };
dq_status dq_calib_set_objective(dq_calib_t* h, int32_t objective, int32_t bits);

/* Which orthogonal optimiser updates the rotation.
 *   DQ_ORTH_QR (default): QR-Orth (Sec. 4.3): a free latent Z with R = the orthogonal factor of Z.
 *   DQ_ORTH_CAYLEY: Cayley SGD with momentum (Algorithm 3), the optimiser Sec. 5.3 and Table 4
 *     compare QR-Orth with.  The iterate is the rotation itself (X_1 = the orthogonal factor of the
 *     current latent, computed once); each dq_calib_step iteration computes the same loss and
 *     dL/dR as QR-Orth and then
 *       M <- beta M - dL/dR;  What = M R^T - R (R^T M R^T) / 2;  W = What - What^T;  M <- W R;
 *       a = min(lr, 2 q / (|W|_F + 1e-8));  Y^0 = R + a M;  Y^i = R + a/2 W (R + Y^(i-1)), i = 1..s;
 *       R <- Y^s
 *     with lr the handle's learning rate, six d x d tensor-core products per iteration.  The
 *     skew-symmetrisation is read as What - What^T and the norm as the Frobenius norm (Algorithm 3
 *     prints W on both sides of that step and does not name the norm).  q <= 0 selects 0.5, s <= 0 selects 2.
 *     The latent Z, the QR method and dq_calib_set_optimizer's choice are not used in this mode;
 *     dq_calib_get_rotation returns the iterate.  Selecting a method resets the momentum, and the
 *     next step starts again from the orthogonal factor of the latent.
 * Errors: INVALID_ARG (bad enum, beta outside [0, 1), q > 1, s > 16), UNSUPPORTED (fp32 path or
 * d == 128: only the tensor-core path with d >= 256 implements it), ALLOC, CUDA. */
enum { DQ_ORTH_QR = 0, DQ_ORTH_CAYLEY = 1 };
dq_status dq_calib_set_orth_method(dq_calib_t* h, int32_t method, float beta, float q, int32_t s);

/* Checkpoint / resume of the optimised parameter (Algorithm 1: Z <- Z0).  dq_calib_set_latent clears
 * the status word. */
dq_status dq_calib_get_latent(dq_calib_t* h, float* d_Z_out);
dq_status dq_calib_set_latent(dq_calib_t* h, const float* d_Z);

/* Synchronises the stream and returns the device status word
 * (DQ_OK / DQ_ERR_SINGULAR / DQ_ERR_NONFINITE / DQ_ERR_TIMEOUT / DQ_ERR_NOT_CONVERGED) or DQ_ERR_CUDA. */
dq_status dq_calib_status(dq_calib_t* h);

/* Failure detection self-test (no counterpart in the paper).  Every wait inside the tensor-core kernels (on
 * a TMA copy, an MMA, the other CTA of a pair) is bounded: when it runs out the kernel records
 * DQ_ERR_TIMEOUT in the status word and returns normally, and from then on the update kernels leave the
 * latent untouched.  This call runs that same wait, with a limit of limit_ns nanoseconds (1 .. 1e8), in a
 * one-thread kernel on a barrier that nothing ever arrives at, with no copy or MMA in flight.  Afterwards
 * dq_calib_status returns DQ_ERR_TIMEOUT and steps leave the latent unchanged until dq_calib_set_latent (or a
 * dq_calib_set_* call) clears the status.  d_waited_ns (nullable, device) receives the time waited.
 * Tensor-core path only (DQ_ERR_UNSUPPORTED otherwise). */
dq_status dq_calib_selftest_bounded_wait(dq_calib_t* h, uint64_t limit_ns, uint64_t* d_waited_ns);

/* Phase times of the most recent dq_calib_step call, averaged per step, in ms
 * (synchronises).  Order: DQ_PHASE_*.  Writes min(n, DQ_PHASE_COUNT) entries
 * of the HOST array ms_by_phase. */
enum {
  DQ_PHASE_QR_FORWARD = 0, /* factorisation, forming R, gauge, operand copies   */
  DQ_PHASE_ROTATE_WHIP = 1, /* O = X R with the fused Eq. 4 epilogue + loss reduce */
  DQ_PHASE_GRAD_ROTATION = 2, /* Gq = X^T G                                      */
  DQ_PHASE_QR_BACKWARD = 3,
  DQ_PHASE_UPDATE = 4,
  DQ_PHASE_COUNT = 5
};
dq_status dq_calib_get_timings(dq_calib_t* h, float* h_ms_by_phase, int32_t n);
/* Enable (1) / disable (0) per-phase CUDA-event timing inside dq_calib_step. */
dq_status dq_calib_set_timing(dq_calib_t* h, int32_t enabled);

/* Read-only views of the handle's device workspaces after a step, for tests and
 * diagnostics.  *d_ptr is valid until the handle is destroyed. */
enum {
  DQ_BUF_R = 0,        /* fp32 [batch][d][d]  rotation used by the last step       */
  DQ_BUF_U = 1,        /* fp32 [batch][d][d]  upper factor, positive diagonal (after incremental steps on the tensor-core
                          path only U^-1 is carried: for d >= 256 it is inverted on demand, to about 1e-5; for d == 128 the
                          view is DQ_ERR_UNSUPPORTED until the next Householder factorisation) */
  DQ_BUF_GQ = 2,       /* fp32 [batch][d][d]  dL/dR                                */
  DQ_BUF_GZ = 3,       /* fp32 [batch][d][d]  dL/dZ                                */
  DQ_BUF_G = 4,        /* dL/dO without the 1/N factor: fp32 [batch][N][d] (fp32 path)
                          or bf16 channel-major [batch][d][N] (tensor-core path)   */
  DQ_BUF_PARTIALS = 5, /* fp32 loss partial sums of the last step, a fixed number per problem: one set per
                          output tile (d = 128 on the tensor-core path: per range of token tiles that one
                          CTA covers; entries no CTA writes stay zero)             */
  DQ_BUF_Z = 6,        /* fp32 [batch][d][d]  current latent                       */
  DQ_BUF_OPT_M = 7,    /* fp32 [batch][d][d]  first moment / velocity (NULL for DQ_SGD)  */
  DQ_BUF_OPT_V = 8,    /* fp32 [batch][d][d]  second moment (DQ_ADAM only)         */
  DQ_BUF_CAYLEY_M = 9, /* fp32 [batch][d][d]  momentum of DQ_ORTH_CAYLEY            */
  DQ_BUF_CAYLEY_ALPHA = 10 /* fp32 [batch]    step size of the last Cayley iteration */
};
dq_status dq_calib_debug_buffer(dq_calib_t* h, int32_t which, void** d_ptr, int64_t* n_elems);

/* For d == 128 on the tensor-core path both contractions and the Eq. 4 epilogue run in one kernel and
 * dL/dO never leaves the chip, so DQ_BUF_G is not written.  keep != 0 makes that kernel store dL/dO to
 * DQ_BUF_G as well (for inspection and tests; the results of a step do not change).  No effect on
 * other shapes, where DQ_BUF_G is always written. */
dq_status dq_calib_set_keep_gradient(dq_calib_t* h, int32_t keep);

/* Number of kernels this library launched through the handle so far. */
int64_t dq_calib_launch_count(dq_calib_t* h);

/* bf16 tensor-core flops the handle's tcgen05 kernels were asked to issue so far (2 m n k per MMA
 * product, three products per split-bf16 term, k clipped to the non-zero blocks of triangular
 * operands exactly as the kernels clip it; counted on the host at launch).  For measurement:
 * the difference across a timed region divided by its duration is the issued MMA rate. */
double dq_calib_mma_flops(dq_calib_t* h);

/* For measurement: times (CUDA events on the handle's work stream; synchronises) `reps` launches of one
 * dense d x d x d product of the kind QR-Orth is made of, on the handle's own operand copies, result to
 * scratch: nterms = 3 on split-bf16 operands (three bf16 MMAs per product term, 6 d^3 MMA flops for the
 * 2 d^3 of the product), nterms = 1 on plain bf16 operands.  *h_ms receives the mean per launch.  Tensor-core
 * path with d >= 256 only; call it after at least one step.  Changes no state of the calibration. */
dq_status dq_calib_time_product(dq_calib_t* h, int32_t nterms, int32_t reps, float* h_ms);

const char* dq_status_string(dq_status s);
void dq_calib_destroy(dq_calib_t* h);

/* Compile-time facts of the loaded library: returns a static string such as
 * "dartquant-b200 sm_100a". */
const char* dq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DARTQUANT_H_ */
