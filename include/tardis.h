/*
 * libtardis — C ABI of the partially linear FFN forward (TARDIS, arXiv 2501.10054)
 * for NVIDIA B200 (sm_100a).
 *
 * The paper's system has an offline part that turns an FFN (weights W1, W2, a
 * per-neuron linear range and linear fit, a compressed copy of W1 used as a
 * predictor) into a constant-folded matrix (Section 5.2, Section 5.3), and an
 * online part that maps an FFN input to the FFN output by speculative
 * approximation and result fixing (Section 5.4).  tardis_fold is the offline
 * part, tardis_ffn_forward the online part, tardis_stats the paper's
 * memory-footprint accounting (Section 5.4, "Memory Footprint") plus run
 * counters.
 *
 * Notation.  The paper writes row vectors, FFN(x) = sigma(x W1) W2 with neuron n
 * = column n of W1 and row n of W2.  This interface takes the nn.Linear storage
 * layout: W1[d_ff, d_model] (row j = neuron j) and W2[d_model, d_ff] (column j
 * = neuron j); W_f = W2 diag(a) W1 is then the transpose of the paper's C and
 * b_f = W2 (a .* b1 + c) + b2 is the paper's B.  (a_j, c_j) are the paper's
 * slope and intercept, [lo_j, hi_j) its half-open range [l1, l2) (Section 5.1.1).
 *
 * All pointers named "device" are CUDA device pointers of the current device;
 * no argument is a host array unless it says so.  No function throws, aborts
 * or prints; every failure is a status code.  A handle is not thread-safe;
 * distinct handles are independent.
 */
#ifndef TARDIS_H_
#define TARDIS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tardis_handle_s* tardis_handle_t;   /* opaque; owns device memory */
typedef void* tardis_stream_t;                      /* a cudaStream_t (0 = default stream) */

typedef enum {
  TARDIS_OK = 0,
  TARDIS_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, negative size, bad enum */
  TARDIS_ERR_UNSUPPORTED = 2,   /* valid request the library has no kernel for (see tardis_fold) */
  TARDIS_ERR_ALLOC = 3,         /* device allocation failed */
  TARDIS_ERR_CUDA = 4,          /* a CUDA call failed; text via tardis_last_error */
  TARDIS_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out */
  TARDIS_ERR_CORRUPT = 6        /* handle magic / guard words damaged */
} tardis_status_t;

typedef enum { TARDIS_F32 = 0, TARDIS_BF16 = 1 } tardis_dtype_t;
/* TARDIS_ACT_RELU: max(z, 0), the activation of the OPT model in the paper's evaluation (Section 7.1). */
typedef enum { TARDIS_ACT_GELU_TANH = 0, TARDIS_ACT_GELU_ERF = 1, TARDIS_ACT_RELU = 2 } tardis_act_t;

/* Inputs of the offline fold.  Every array is read on `stream` during
 * tardis_fold and copied or transformed into handle-owned memory; once that
 * stream has drained the caller may free all of them. */
typedef struct {
  int32_t d_model;            /* d; multiple of 8 and of pred_group                       */
  int32_t d_ff;               /* h; multiple of 32                                        */
  int32_t dtype;              /* tardis_dtype_t: type of W1, W2, pred_scale, x and y      */
  int32_t act;                /* tardis_act_t                                             */
  const void* W1;             /* device [d_ff, d_model] row-major; row j = neuron j       */
  const void* W2;             /* device [d_model, d_ff] row-major; column j = neuron j    */
  const float* b1;            /* device [d_ff]    or NULL (= 0)                           */
  const float* b2;            /* device [d_model] or NULL (= 0)                           */
  const float* lo;            /* device [d_ff]; neuron j is in range iff lo <= z < hi     */
  const float* hi;            /* device [d_ff]                                            */
  const float* a;             /* device [d_ff]; linear fit a*z + c on the range           */
  const float* c;             /* device [d_ff]                                            */
  int32_t pred_bits;          /* bits per predictor code: 2 (the paper's setting, Section 6;
                                 every path), 3 or 4 (batched and generic paths; 3 needs
                                 d_model % 32 == 0) or 8 (generic kernels only); the paper
                                 sweeps this size in Section 7.6                           */
  int32_t pred_group;         /* G: channels per quantisation group; multiple of 16       */
  const uint32_t* pred_codes; /* device [d_ff, d_model*pred_bits/32]: row j is one bit stream
                                 over its words, lowest bits first; channel k holds its bits
                                 [pred_bits k, pred_bits (k + 1)) (word pred_bits k / 32,
                                 from bit pred_bits k % 32 upwards; with 2, 4 or 8 bits a
                                 code stays inside one word, a 3-bit code may go on in the
                                 lowest bits of the next word)                            */
  const void* pred_scale;     /* device [d_ff, d_model/G], type `dtype`                   */
  const uint8_t* pred_zero;   /* device [d_ff, d_model/G], integer zero-point 0..2^pred_bits-1 */
  uint32_t flags;             /* 0, or one of the TARDIS_FOLD_* study modes below          */
} tardis_fold_desc_t;

/* Study modes of the fold for bf16 layers (tardis_fold_desc_t.flags), after the paper's look at the precision of
 * the reordered product (Section 7.7): 0 folds through the tensor cores with diag(a) W1 held as the exact sum of two
 * bf16 matrices and fp32 accumulation (the default); TARDIS_FOLD_BF16_INTERMEDIATE keeps only the leading bf16 term
 * of diag(a) W1 (the "bf16 intermediate" row of the paper's table); TARDIS_FOLD_FP32_PLAIN computes the product with
 * plain fp32 arithmetic from the fp32 values of a W1 (no tensor cores).  All three round W_f to bf16 once at the end. */
#define TARDIS_FOLD_BF16_INTERMEDIATE 1u
#define TARDIS_FOLD_FP32_PLAIN 2u

/* Counters and sizes.  Byte counts are the resident state of the handle,
 * following the paper's footprint components: folded matrix + bias, predictor,
 * original weights kept for fixing (here: all of W1 and W2^T, any neuron can
 * be flagged), per-neuron tables, scratch. */
typedef struct {
  uint64_t calls;               /* tardis_ffn_forward / tardis_ffn_forward_static calls that launched work */
  uint64_t tokens;              /* tokens processed                                        */
  uint64_t flagged_total;       /* sum over tokens of flagged neurons                      */
  uint64_t flagged_max;         /* largest flagged count of a single token                 */
  uint64_t last_path;           /* 0 none, 1 generic kernels, 2 fused decode kernel, 3 batched/prefill,
                                   5 generic kernels on the library's built-in scratch
                                   (tardis_ffn_forward_static)                              */
  uint64_t bytes_folded;        /* W_f and b_f                                             */
  uint64_t bytes_predictor;     /* codes + scales + zero-points as stored                  */
  uint64_t bytes_tables;        /* lo, hi, a, c, b1                                        */
  uint64_t bytes_w1;
  uint64_t bytes_w2t;
  uint64_t bytes_scratch;
  uint64_t device_error;        /* sticky device-side error word, 0 = none                 */
  uint64_t exact_rechecks;      /* predictor scores re-evaluated by the exact slow path    */
  uint64_t launches;            /* kernels launched by tardis_ffn_forward so far           */
  uint64_t last_union;          /* neurons flagged by at least one token of the most recent
                                   launch of the fused decode kernel (the rows it fetched)   */
} tardis_stats_t;

/* Offline part (Section 5.2 constant folding, Section 5.3 predictor set-up).
 * Computes W_f = W2 diag(a) W1 and b_f = W2 (a .* b1 + c) + b2 with accumulation
 * in at least fp32 and one rounding to `dtype`, stores W2 transposed, keeps a
 * copy of W1 and of the predictor.  Asynchronous on `stream` after the device
 * allocations; *out is valid on return with TARDIS_OK.
 * Errors: INVALID_ARG (NULL desc/out/required array, pointer not 16-byte
 * aligned, d_model % 8, d_model % pred_group, pred_group % 16, d_ff % 32,
 * non-positive sizes, unknown enum, pred_bits outside 1..8), UNSUPPORTED (pred_bits of 1, 5, 6 or 7), ALLOC, CUDA.
 * Forward calls on the handle must be ordered after `stream` (same stream, or an event): the fold is asynchronous. */
tardis_status_t tardis_fold(const tardis_fold_desc_t* desc, tardis_stream_t stream,
                            tardis_handle_t* out);

/* Online part (Section 5.4): y[t,:] = W_f x[t,:] + b_f
 *      + sum over neurons j flagged for token t of W2[:,j] (GELU(z_j) - a_j z_j - c_j),
 * z_j = W1[j,:] x[t,:] + b1_j recomputed from the original row; neuron j is
 * flagged for token t when the predictor score
 *      zhat = b1_j + sum_g scale[j,g] sum_{k in g} (code[j,k] - zero[j,g]) x[t,k]
 * is not in [lo_j, hi_j) (NaN counts as outside).
 * x, y: device [n_tokens, d_model] row-major in the handle's dtype, 16-byte
 * aligned, not overlapping; y is fully overwritten.  Asynchronous on `stream`,
 * allocates nothing, does not synchronise.  n_tokens == 0 returns TARDIS_OK
 * without launching.  The kernel path depends on n_tokens and the handle only.
 * Calls on one handle must be stream-ordered with respect to each other (they
 * share the handle's scratch).
 * Errors: INVALID_ARG (NULL/destroyed handle, NULL or misaligned x/y,
 * n_tokens < 0, the handle's device is not the current device), CUDA. */
tardis_status_t tardis_ffn_forward(tardis_handle_t handle, const void* x, void* y,
                                   int64_t n_tokens, tardis_stream_t stream);

/* The online part for callers that must not allocate device memory.  (The paper has no counterpart of
 * this call; it exists for the way this library gets embedded.)  Some hosts of this code cannot go
 * to the CUDA allocator once they are running: a serving process that handed all device memory to
 * its own pool at start-up, a control loop with a "no driver allocation after initialisation" rule,
 * code that runs while a stream is being captured.  tardis_ffn_forward already takes its scratch
 * from the handle; this variant takes it from neither the handle nor the allocator: the fp32 output
 * accumulator and the flag bitmap of the call live in a fixed 4 MiB array that is part of the
 * library image (every GPU that loads the library holds those 4 MiB until the process exits).  It
 * calls no cudaMalloc, cudaFree or other allocating routine.
 * Same arguments, result and error behaviour as tardis_ffn_forward, computed by the generic
 * kernels (the exact-range mode of tardis_set_path(handle, 4) is honoured; the other path choices do
 * not apply), with these differences:
 *   - n_tokens <= 64 and n_tokens * (4 * d_model + d_ff / 8) <= 4 MiB (each of the two terms rounded
 *     up to 256 bytes), else TARDIS_ERR_UNSUPPORTED with the reason in tardis_last_error; the
 *     handle's device must be the current device, else TARDIS_ERR_INVALID_ARG;
 *   - the first call on a device asks the runtime for the array's device address
 *     (cudaGetSymbolAddress, under a lock) and keeps it; make that first call before any stream
 *     capture starts, and do not reset the device (cudaDeviceReset) while the library is loaded:
 *     the kept address would be stale;
 *   - the array is shared by every call and every handle in the process and keeps what the last
 *     call left in it.  A call overwrites all of the part it uses before reading it, so stale
 *     contents are harmless, but two calls that overlap in time on the GPU (different streams, or
 *     one of them tardis_ffn_forward_static and the other any work still using the array) race:
 *     order them on one stream or with events. */
tardis_status_t tardis_ffn_forward_static(tardis_handle_t handle, const void* x, void* y,
                                          int64_t n_tokens, tardis_stream_t stream);

/* The dense product every batched step of the path is made of, on its own: C = A B^T with bf16 operands
 * and fp32 accumulation on the tensor cores (the batched speculative product X W_f^T of Section 5.4, the
 * fold W2 (diag(a) W1) of Section 5.2 and the batched pre-activations X W1^T all have this shape).
 * A: device bf16 [M, K] row-major with leading dimension lda; B: device bf16 [N, K] row-major (ldb);
 * C: device float [M, N] (ldc), fully overwritten.  K, lda, ldb multiples of 8; A, B and C 16-byte aligned
 * (a view that starts at an odd column is refused).
 * Asynchronous on `stream`.  Errors: INVALID_ARG, UNSUPPORTED (driver without tensor-map support), CUDA. */
tardis_status_t tardis_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int32_t lda,
                                 const void* B, int32_t ldb, float* C, int32_t ldc, tardis_stream_t stream);

/* Synchronises the stream of the handle's most recent call, then fills *out
 * (host memory).  Returns TIMEOUT / CORRUPT when the device error word says so. */
tardis_status_t tardis_stats(tardis_handle_t handle, tardis_stats_t* out);

/* Debug capture for parity checks: when set, every later forward call also
 * writes, for its tokens, the flag bitmap (device uint32 [n_tokens, d_ff/32],
 * bit j%32 of word j/32 = neuron j flagged) and/or the predictor scores as the
 * kernel decided on them (device double [n_tokens, d_ff]).  Either may be NULL;
 * both NULL switches capture off.  The buffers must cover the largest n_tokens
 * passed while capture is on. */
tardis_status_t tardis_set_debug_capture(tardis_handle_t handle, uint32_t* flag_bitmap,
                                         double* scores);

/* Copies the folded state out for inspection: Wf device [d_model, d_model]
 * row-major in the handle's dtype (row i = output channel i, i.e. W_f itself,
 * the transpose of the paper's C), bf device float [d_model].  Either may be NULL. */
tardis_status_t tardis_export_folded(tardis_handle_t handle, void* Wf, float* bf,
                                     tardis_stream_t stream);

/* Offline statistics of one layer: the range and the linear function of every
 * neuron from calibration pre-activations.  The paper picks, per neuron, the
 * input range that holds a given portion of the profiled activation inputs and
 * fits y = a z + c to the activation inside it by least squares (the procedure is
 * described with Insight 2 in Section 4.1; steps 2 and 3 of the list in Section 5.1;
 * Section 5.1.1 for the single range and its linear function).  Here the range is
 * the one between the quantiles q_lo and q_hi of the neuron's samples (linear
 * interpolation between the order statistics around position q (n_cal - 1),
 * evaluated in double precision, stored in single); the fit is ordinary least
 * squares of GELU(z) on z over the samples with lo <= z < hi, in double
 * precision; a neuron with fewer than two samples in range (or in-range
 * variance below 1e-30) takes the tangent of GELU at (lo + hi) / 2.
 *   z      device [d_ff, n_cal] float, row j = samples of neuron j, leading
 *          dimension ldz >= n_cal (e.g. the output of tardis_gemm_bf16 with
 *          A = W1, B = calibration tokens); samples must be finite
 *   b1     device [d_ff] added to the samples, or NULL
 *   lo, hi, a, c   device [d_ff] float, outputs (what tardis_fold takes)
 * 1 <= n_cal <= 8192 (TARDIS_ERR_UNSUPPORTED beyond), 0 <= q_lo <= q_hi <= 1.
 * Asynchronous on `stream`; allocates nothing; nothing is kept. */
tardis_status_t tardis_calibrate(int32_t d_ff, int32_t n_cal, const float* z, int64_t ldz, const float* b1,
                                 double q_lo, double q_hi, int32_t act, float* lo, float* hi, float* a, float* c,
                                 tardis_stream_t stream);

/* The range search of Algorithm 1 (Section 5.1.1, "Range Searching") for every neuron of one layer, from the same
 * calibration pre-activations as tardis_calibrate: the range starts empty at the centroid of the neuron's samples (the
 * sample with the highest Gaussian kernel density estimate; kernel width 1.06 std n_cal^(-1/5), the paper names neither
 * kernel nor width) and grows by `step` at a time on the side whose grown range has the smaller approximation error (mean
 * squared residual of the least-squares line over the samples inside; the right side on a tie; a side that has passed the
 * outermost sample is not grown) until the share of the samples with lo <= z < hi reaches the neuron's threshold; then the
 * line of the final range is fitted as in tardis_calibrate.  The listing's left candidate reads (R.left - s, R.left);
 * it is taken as (R.left - s, R.right).  Bounds are centroid - k_left step and centroid + k_right step, evaluated in
 * double precision and stored in single.
 *   thresholds   device [d_ff] float, the per-neuron coverage t of Section 5.1.1's neuron-level thresholds, or NULL: then
 *                every neuron uses `threshold`
 *   steps_taken  device [d_ff] int32 or NULL: number of growth steps per neuron
 * 1 <= n_cal <= 2048 (TARDIS_ERR_UNSUPPORTED beyond), step > 0, thresholds in [0, 1].  Other arguments as in
 * tardis_calibrate.  Asynchronous on `stream`; allocates nothing; nothing is kept. */
tardis_status_t tardis_range_search(int32_t d_ff, int32_t n_cal, const float* z, int64_t ldz, const float* b1,
                                    const float* thresholds, double threshold, double step, int32_t act, float* lo, float* hi,
                                    float* a, float* c, int32_t* steps_taken, tardis_stream_t stream);

/* The neuron-level thresholds of Section 5.1.1: within a layer, the layer's threshold t_layer is distributed over the
 * neurons by minimising sum_j E_j t_j subject to sum_j t_j = t_layer d_ff, where E_j is the error contribution of neuron j.
 * As printed the problem has no bounds on t_j and no minimum; it is read with the box t_min <= t_j <= t_max, whose solution
 * is: every neuron gets t_min, and the remaining budget (t_layer - t_min) d_ff goes, t_max - t_min each, to the neurons in
 * order of increasing E_j (the smaller index first among equal errors); at most one neuron ends between the bounds.  E_j is
 * measured as Algorithm 1's approx_error does: the mean squared residual of the least-squares line over the neuron's
 * calibration samples inside its range [lo_j, hi_j) (0 with fewer than two samples inside), in double precision, stored in
 * single; the order is taken on the stored values.
 *   z, ldz, b1, n_cal   as in tardis_range_search (n_cal <= 2048);  lo, hi   device [d_ff], e.g. a search at t_layer;
 *   err         out, device [d_ff]: E_j;   thresholds   out, device [d_ff]: t_j, what tardis_range_search takes next.
 * 0 <= t_min <= t_layer <= t_max <= 1.  Asynchronous on `stream`; allocates nothing; nothing is kept. */
tardis_status_t tardis_neuron_thresholds(int32_t d_ff, int32_t n_cal, const float* z, int64_t ldz, const float* b1,
                                         const float* lo, const float* hi, int32_t act, double t_layer, double t_min,
                                         double t_max, float* err, float* thresholds, tardis_stream_t stream);

/* Chooses the kernel path: 0 = automatic (default), 1 = always the generic
 * kernels, 2 = the fused decode kernel for every token count up to 4096 (in
 * launches of at most 4 tokens; layers it does not serve fall back as in 0),
 * 3 = the batched tensor-core path for every token count (bf16
 * layers; other layers fall back to the generic kernels), 4 = the generic
 * kernels with the range check taken on the true pre-activations
 * z = W1 x + b1 instead of the predictor's scores: the paper's third scenario
 * of Section 7.7, which takes the predictor out of the result to show its
 * effect (the debug capture then holds z).  For testing one path against the
 * other. */
tardis_status_t tardis_set_path(tardis_handle_t handle, int32_t path);

/* Deterministic accumulation, on (1) or off (0, the default).  The paper does not
 * say in which order the speculative product and the corrections of Section 5.4
 * are added up; by default this library adds partial sums to y in the order in
 * which the CTAs finish (floating-point atomics), so the last bits of y may differ
 * between two runs on the same input.  With the mode on, every partial sum is
 * written to a place of its own and added in one fixed order (the fused decode
 * kernel keeps [d_model / 256 + CTAs][4][d_model] fp32 partial outputs, allocated
 * by this call the first time, and a second small kernel sums them; the batched
 * products no longer split their channel range): y is then the same bits from run
 * to run for the same handle, input and token count.  Flags do not depend on the
 * mode.  Cost: one more launch per 4 tokens on the fused path, and products of
 * few tokens run on fewer CTAs on the batched path.
 * Returns TARDIS_ERR_UNSUPPORTED when the layer is served only by kernels that
 * add with atomics (fp32 layers, 8-bit codes, wider bf16 layers on the per-token
 * kernel); a later tardis_ffn_forward on a handle in this mode returns
 * TARDIS_ERR_UNSUPPORTED too where its path choice (tardis_set_path 1 or 4) leads
 * to such kernels.  tardis_ffn_forward_static does not look at the mode. */
tardis_status_t tardis_set_deterministic(tardis_handle_t handle, int32_t on);

/* Offline: the predictor of a layer, built on the GPU.  The paper obtains its predictor by GPTQ with 2-bit precision
 * (Section 6; Section 5.3 for what the predictor is, Section 7.6 for other widths).  Per neuron, channels in ascending
 * order: when channel k opens a group, the group's grid is taken from the weights as they are then (range widened to
 * contain 0; scale = (max - min) / (2^bits - 1) rounded to `dtype`, 1 if that is 0; zero-point = round(-min / scale)
 * clamped to the code range); q_k = clip(round(w_k / scale + zero)); e_k = (w_k - scale (q_k - zero)) / U[k][k]; every
 * later channel takes w_j <- w_j - e_k U[k][j].  Rounding is to nearest-even, all arithmetic is double precision with
 * separately rounded products and differences, so the codes are those of a plain double-precision implementation.
 *   W1     device [d_ff, d_model] row-major in `dtype`;
 *   U      device double [d_model, d_model] row-major, the upper Cholesky factor of the inverse Hessian of the layer's
 *          inputs (U^T U = H^-1, H = (2/N) X^T X plus damping: made by the caller, e.g. with a library Cholesky), only
 *          its upper triangle is read; NULL = identity, which gives plain rounding to nearest;
 *   bits   2, 3, 4 or 8; group a multiple of 64 that divides d_model;
 *   codes  out, device [d_ff, d_model bits / 32] (one bit stream per row, channel order ascending, lowest bits first);
 *   scale  out, device [d_ff, d_model / group] in `dtype`; zero out, device bytes of the same shape.
 * The outputs are what tardis_fold_desc_t takes as pred_codes, pred_scale, pred_zero.  The call allocates its scratch
 * (8 d_ff d_model bytes and a little more), runs on `stream` and returns after the stream has finished the work.
 * Errors: INVALID_ARG, ALLOC, CUDA. */
tardis_status_t tardis_build_predictor(int32_t d_ff, int32_t d_model, tardis_dtype_t dtype, const void* W1, const double* U,
                                       int32_t bits, int32_t group, uint32_t* codes, void* scale, uint8_t* zero,
                                       tardis_stream_t stream);

/* A chain of layers on one residual stream.  The paper replaces the FFN block inside an existing
 * model (Section 6) and has no call of this kind; this is the shape in which a decoder hands the
 * FFN blocks of consecutive layers to the library, attention left out:
 *     s_0 = x;   u_l = normalise ? LayerNorm_l(s_l) : s_l;   f_l = FFN_l(u_l)  (tardis_ffn_forward);
 *     s_{l+1} = residual ? s_l + f_l : f_l;   y = s_{n_layers}.
 * LayerNorm_l(v)[i] = (v[i] - mean(v)) / sqrt(var(v) + ln_eps) * gamma_l[i] + beta_l[i], mean and
 * variance (divisor d_model) over the token's row, computed in fp32 and rounded to the layers' dtype;
 * s_l + f_l is added in fp32 and rounded to the dtype once per layer.
 *   layers    host array of n_layers handles of the same d_model, dtype and device (each keeps its own
 *             path choice, capture and accumulation mode);
 *   ln_gamma, ln_beta   host arrays of n_layers device pointers to [d_model] fp32, or NULL (1 and 0);
 *   x, y      device [n_tokens, d_model] in the layers' dtype, 16-byte aligned; y may be x (in place);
 *   work      device scratch of at least 2 n_tokens d_model elements, caller-owned (the call allocates
 *             nothing); ignored when keep is given;
 *   keep      NULL, or device [n_layers][2][n_tokens, d_model]: u_l and f_l of every layer stay there
 *             for the caller to look at (tests compare each layer with the oracle on that layer's input).
 * Everything is enqueued on `stream`; d_model up to 12288.  Errors: INVALID_ARG for a bad descriptor,
 * mismatched layers, a missing or small buffer; otherwise what tardis_ffn_forward returns. */
typedef struct {
  int32_t n_layers;
  const tardis_handle_t* layers;
  int32_t normalise;               /* 1: layer normalisation before every layer */
  const float* const* ln_gamma;
  const float* const* ln_beta;
  float ln_eps;
  int32_t residual;                /* 1: s_{l+1} = s_l + f_l; 0: s_{l+1} = f_l */
} tardis_stack_desc_t;
tardis_status_t tardis_stack_forward(const tardis_stack_desc_t* desc, const void* x, void* y, void* work, size_t work_bytes,
                                     void* keep, size_t keep_bytes, int64_t n_tokens, tardis_stream_t stream);

/* Profiling aid of the fused decode kernel (the online path of Section 5.4 as one launch).  A library
 * built with -DTARDIS_PHASE_STAMPS (python -m paper_2501_10054_b200.build --stamps) makes every CTA of that
 * kernel record the GPU's global nanosecond timer at its phase boundaries; this call synchronises the
 * device and copies the table of the most recent launch to `stamps`, HOST memory of max_ctas x 16 int64:
 * per CTA, slot 0 kernel entry, 1 x loaded, 2 fixed-point x ready, 3 predictor done (first predictor
 * warp), 4 folded product done (first streaming warp), 5 flagged list complete, 6 result fixing done,
 * 7 CTA counted as finished, 8 y written (last CTA only, else 0), 9 the CTA's number of flagged neurons
 * (a count, not a time); CTAs beyond the grid stay 0.  The ordinary build returns TARDIS_ERR_UNSUPPORTED
 * and its kernel carries no stamps.  Errors: INVALID_ARG (NULL, max_ctas <= 0), UNSUPPORTED, CUDA. */
tardis_status_t tardis_debug_phase_stamps(long long* stamps, int32_t max_ctas);

/* A handle's state in a binary file and back (Section 6: the offline component writes the folded matrix and the
 * predictor to a binary file that the runtime loads).  tardis_save synchronises the handle's last stream and writes, to
 * the HOST path `path`: a 64-byte header (magic "TARDIS01", d_model, d_ff, dtype, act, pred_group, pred_bits), then W1,
 * W2^T, the folded matrix (as stored: [channel][output]), b_f, lo, hi, a, c, b1, the predictor codes, scales and
 * zero-points as raw little-endian arrays, then a 64-bit FNV-1a checksum of the array bytes.  tardis_load reads such a
 * file, allocates a handle on the current device, uploads the arrays and derives the kernel-specific copies as
 * tardis_fold does; no fold is recomputed, so the loaded handle gives bit-identical flags and scores, and outputs equal
 * to those of the saved handle up to the order of floating-point reductions.  *out is valid on return with TARDIS_OK;
 * work is enqueued on `stream`.  Errors: INVALID_ARG (NULL, file cannot be opened or written), CORRUPT (bad magic,
 * implausible header, truncated file, checksum mismatch), ALLOC, CUDA. */
tardis_status_t tardis_save(tardis_handle_t handle, const char* path);
tardis_status_t tardis_load(const char* path, tardis_stream_t stream, tardis_handle_t* out);

/* Every wait inside the kernels (on a bulk copy's barrier) is bounded: when the limit runs out the kernel records it in
 * the handle's device error word, skips the work that needed the data and returns; tardis_stats then reports
 * TARDIS_ERR_TIMEOUT until the word is cleared.  tardis_debug_wait_timeout makes exactly that happen on purpose, for
 * testing the reporting path without any fault: it launches one warp that waits, for at most limit_cycles SM clock
 * cycles (0 .. 2e9), on a barrier whose bytes never arrive.  tardis_clear_error synchronises the handle's last stream and
 * resets the error word.  (The paper has no counterpart of these two calls.)  Errors: INVALID_ARG, CUDA. */
tardis_status_t tardis_debug_wait_timeout(tardis_handle_t handle, int64_t limit_cycles, tardis_stream_t stream);
tardis_status_t tardis_clear_error(tardis_handle_t handle);

/* For testing what the library does when the device allocator says no, without exhausting a GPU: after this call the next
 * `nth` device allocations of the library (process-wide, any thread) succeed and the one after them fails once, as
 * cudaMalloc would with no memory left; nth < 0 switches the injection off.  The entry point that hits the failure
 * returns TARDIS_ERR_ALLOC and must leave nothing allocated behind.  (The paper has no counterpart of these two calls.) */
tardis_status_t tardis_debug_fail_alloc(int32_t nth);
/* How many device allocations of the library are alive in this process, and their bytes (guard areas not counted): what a
 * test compares before and after a failed call. */
tardis_status_t tardis_debug_live_allocations(int64_t* count, int64_t* bytes);

/* Every device buffer a handle owns lies between two guard areas of 256 bytes holding a fixed pattern; tardis_stats reads
 * the guards of the handle's buffers back and returns TARDIS_ERR_CORRUPT (device_error = 2) when one has changed, i.e. when
 * some kernel wrote past an end of a buffer.  tardis_debug_damage_guard changes (repair = 0) or restores (repair = 1) the
 * four guard bytes in front of (front = 1) or behind (front = 0) the handle's fp32 accumulator, so that this report can be
 * tested; the write stays inside the allocation and faults nothing.  (The paper has no counterpart of this call.) */
tardis_status_t tardis_debug_damage_guard(tardis_handle_t handle, int32_t front, int32_t repair);

/* Frees everything the handle owns (synchronises the device first). */
tardis_status_t tardis_destroy(tardis_handle_t handle);

const char* tardis_status_string(tardis_status_t status);
/* Text of the most recent CUDA error seen by this thread in the library ("" if none). */
const char* tardis_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TARDIS_H_ */
