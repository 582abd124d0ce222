/*
 * fp8lin.h -- C ABI of the B200 (sm_100a) FP8 linear layer with dynamically
 * updated per-tensor scaling bias, after "Training and inference of large
 * language models using 8-bit floating point" (arXiv 2309.17224).
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 *  - Every call returns an fp8_status_t.  Nothing throws, nothing is printed
 *    and no environment variable is read.
 *  - All tensor pointers are DEVICE pointers owned by the caller; the library
 *    never allocates, frees or retains them.  "d_" marks a device scalar.
 *    The only host pointers are the fp8_ctx handle, `flags` of
 *    fp8_device_flags, the counters of fp8_prediction_stats and
 *    fp8_launch_count, the descriptor array of fp8_cast_group and the
 *    arguments of fp8_scaling_bias_host.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Calls are asynchronous and ordered on that stream like any
 *    kernel launch.  Calls that share one fp8_ctx must be issued from one host
 *    thread at a time, and decode-size matmuls (at most 128 rows of output:
 *    they may split the contraction through the context's workspace) that
 *    share one fp8_ctx must not overlap on the device: keep them on one
 *    stream, or order the streams with events, or use one context per stream.
 *    Inside the library a kernel may be launched so that it starts while the
 *    call before it on the stream is draining; it touches no memory before
 *    that call has completed, so stream order holds as for any launch.
 *  - Tensors are row-major.  X[T,K] activations, W[N,K] weights (the layout of
 *    a PyTorch nn.Linear), dY[T,N] output gradients; Y[T,N], dX[T,K], dW[N,K].
 *  - FP8 bytes are the native Blackwell encodings (Table 7 rows "(b)": E4M3
 *    with exponent bias 7 and max 448, E5M2 with bias 15 and max 57344).
 *    Scaling biases are always the paper-convention integers of Eq. 3.  Under
 *    FP8_CONV_PAPER the E4 shift actually applied is bias+1, because a byte of
 *    the paper's E4 format (Table 7 row "(a)", exponent bias 8, max 240) read
 *    as a native E4M3 byte is exactly twice the value; the matmuls take that
 *    extra factor out again.  Byte c of a tensor with bias b therefore means
 *    native_value(c) * 2^-(b + delta), delta = 1 for (E4, FP8_CONV_PAPER) and
 *    0 otherwise.  Paper E4 codes without a native counterpart: +-240 (emitted
 *    as +-224) and the paper's NaN code 0x80 (natively -0).
 *  - Argument errors are detected on the host and returned BEFORE anything is
 *    launched.  Data-dependent conditions never fail a call; they set sticky
 *    bits in a device status word (see fp8_device_flags).
 */
#ifndef FP8LIN_H
#define FP8LIN_H

#include <stdint.h>

#if defined(__GNUC__)
#define FP8_API __attribute__((visibility("default")))
#else
#define FP8_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FP8_OK = 0,
    FP8_ERR_NULL = 1,           /* a required pointer is NULL */
    FP8_ERR_SHAPE = 2,          /* a dimension is <= 0, or ld < cols */
    FP8_ERR_ALIGN = 3,          /* pointer / leading dimension alignment the kernels need is not met */
    FP8_ERR_DTYPE = 4,          /* enum value out of range */
    FP8_ERR_UNSUPPORTED = 5,    /* valid request that this build has no kernel for (there is no fallback path) */
    FP8_ERR_CUDA = 6,           /* a CUDA runtime / driver call failed (launch, attribute, tensor-map encode) */
    FP8_ERR_DEVICE_TIMEOUT = 7, /* reported by fp8_device_flags when a bounded device-side wait expired */
    FP8_ERR_TOO_LARGE = 8       /* tensor exceeds the fixed workspace of fp8_amax_noalloc */
} fp8_status_t;

typedef enum { FP8_E4 = 0, FP8_E5 = 1 } fp8_format_t;

/* Which max_num Eq. 3 uses: the paper's own formats (240 / 57344) or the
 * native formats' (448 / 57344). */
typedef enum { FP8_CONV_PAPER = 0, FP8_CONV_NATIVE = 1 } fp8_conv_t;

typedef enum { FP8_BF16 = 0, FP8_F16 = 1, FP8_F32 = 2 } fp8_dtype_t;

/* Sticky device status bits. */
#define FP8_FLAG_NONFINITE_AMAX 1u /* an amax was inf or NaN; its bias was set to 0 */
#define FP8_FLAG_ZERO_AMAX 2u      /* an amax was 0; its bias was set to 0 */
#define FP8_FLAG_SATURATED 4u      /* a cast clipped at least one value (finite or infinite) to the format's maximum.
                                    * Under (FP8_E4, FP8_CONV_PAPER) this also fires for a just-in-time FP8-AMAX
                                    * cast whose scaled amax lands in (232, 240]: Eq. 3 places it at or below the
                                    * paper format's 240, the one magnitude code with no native counterpart, and
                                    * the bytes carry 224 instead (about one tensor in twenty; the largest
                                    * elements lose at most 6.7 %).  FP8_CONV_NATIVE never clips a finite
                                    * just-in-time cast. */
#define FP8_FLAG_TIMEOUT 8u        /* a bounded wait inside a kernel expired; that kernel's output is invalid */

typedef struct fp8_ctx fp8_ctx;

/* Create / destroy a context on `device`.  The context owns its device
 * workspace: a status word, reduction slots and a 64 MB FP32 buffer for the
 * partial sums of split-contraction (decode-size) matmuls.  fp8_create is the
 * only call that allocates device memory; it also raises the dynamic
 * shared-memory limit of the matmul kernels.  It must not be called during
 * stream capture.  The context-taking calls that enqueue work (fp8_amax,
 * fp8_scaling_bias, fp8_cast_*, fp8_ptq_weights, fp8_linear_*) neither
 * synchronise nor allocate, so a whole step of them can be captured into a
 * CUDA graph and replayed. */
FP8_API fp8_status_t fp8_create(fp8_ctx **ctx, int device);
FP8_API fp8_status_t fp8_destroy(fp8_ctx *ctx);

FP8_API const char *fp8_status_string(fp8_status_t status);

/* Kernels launched by this library in this process so far (all contexts; host
 * counter, bumped beside every launch; fp8_amax_noalloc is not counted).  The
 * difference of two readings is what a span of calls launched. */
FP8_API fp8_status_t fp8_launch_count(uint64_t *count);

/* Synchronises `stream`, copies the sticky status word to *flags (host) and,
 * if `clear` is non-zero, resets it.  Returns FP8_ERR_DEVICE_TIMEOUT if
 * FP8_FLAG_TIMEOUT was set, else FP8_OK. */
FP8_API fp8_status_t fp8_device_flags(fp8_ctx *ctx, void *stream, unsigned *flags, int clear);

/* Failure-detection self-test (no counterpart in the paper).  Every wait inside the kernels is bounded; this
 * call makes one run out on purpose, without any fault: a one-CTA kernel waits on a barrier that nothing will
 * ever complete, gives up after limit_ns (1 .. 100 000 000), raises FP8_FLAG_TIMEOUT and returns normally.
 * Returns FP8_OK when exactly that happened; fp8_device_flags then reports FP8_ERR_DEVICE_TIMEOUT until the flag
 * is cleared, and the context stays usable.  Synchronises `stream`. */
FP8_API fp8_status_t fp8_selftest_wait_expiry(fp8_ctx *ctx, uint64_t limit_ns, void *stream);

/* Measurement aid (no counterpart in the paper): the tensor-pipe ceiling of the CTA-pair matmul kernel on this
 * device.  Runs that kernel for an M x N x K problem (M > 128) with its operand loads switched off: the shared-memory
 * stages are filled once with a fixed pattern of finite E4M3 bytes and every tcgen05.mma reads them as they stand;
 * barriers, instruction stream, accumulators, epilogue and output stores are those of fp8_linear_fwd.  Timed by the
 * caller with CUDA events, 2 M N K / time is what the kernel would reach if moving operands cost nothing -- the
 * denominator that isolates the operand feed.  `out` [M, N] bf16 (16-byte aligned, N % 8 == 0) receives
 * meaningless values; `d_zero` is a device int32 holding 0 (it stands in for the two biases). */
FP8_API fp8_status_t fp8_selftest_mma_ceiling(fp8_ctx *ctx, void *out, const int32_t *d_zero, int64_t M, int64_t N,
                                              int64_t K, void *stream);

/* amax = max(|x|) over the whole tensor (Eq. 3, first line).
 *   x       [rows, cols] with leading dimension ld (elements), dtype x_dt
 *           (FP8_BF16, FP8_F16 or FP8_F32)
 *   d_amax  out, one float.  NaN if any element is NaN, else the exact maximum
 *           magnitude (inf included).
 * Needs x aligned to its element size only; 16-byte aligned x with ld == cols
 * (or 16-byte aligned rows) takes the vectorised path. */
FP8_API fp8_status_t fp8_amax(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                      float *d_amax, void *stream);

/* amax for callers that cannot allocate device memory (the paper has no
 * counterpart; this exists for deployment).  fp8_amax needs an fp8_ctx, and
 * fp8_create calls cudaMalloc for the reduction workspace.  Programs that have
 * handed all device memory to their own allocator, that must not call
 * cudaMalloc on a serving thread (it synchronises the whole device), or that
 * run as a plug-in without an allocator can use this entry point instead: it
 * takes no context and calls no cudaMalloc, cudaFree or any other allocating
 * routine.  Its workspace is a 32 KiB array inside the library's device image,
 * which every GPU that loads the library holds until the process exits.
 *   x       [rows, cols] bf16, contiguous (ld == cols), 16-byte aligned
 *   d_amax  out, one float, same value as fp8_amax writes
 * Limits and rules:
 *   - at most 2^29 elements (1 GiB of bf16): one partial maximum per
 *     65 536-element chunk, 8192 chunks.  Larger tensors return
 *     FP8_ERR_TOO_LARGE and nothing is launched.
 *   - the first call on each device looks up the array's device address
 *     (with that device current); make that first call before any stream
 *     capture begins.  The launch goes to the current device.
 *   - all calls on a device share the one array: calls whose kernels may
 *     overlap on the GPU (different streams with no ordering between them)
 *     race and give wrong results.  Calls ordered on one stream, or by
 *     events, are safe; each call leaves the array ready for the next. */
FP8_API fp8_status_t fp8_amax_noalloc(const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                                      float *d_amax, void *stream);

/* scaling_bias = floor(log2(max_num / amax)) - margin (Eq. 3, second line;
 * the margin is the one of Section 3.2), evaluated exactly on the bits of
 * amax.  amax == 0 or non-finite gives bias 0 and sets a status flag.
 *   d_amax in, d_bias out: device scalars. */
FP8_API fp8_status_t fp8_scaling_bias(fp8_ctx *ctx, const float *d_amax, fp8_format_t fmt, fp8_conv_t conv,
                              int32_t margin, int32_t *d_bias, void *stream);

/* Amax history (Section 3: where a second pass over memory is too costly, the
 * scale may come from the amax of earlier steps): a ring of the last `len` amax
 * values of one tensor.  The call stores *d_amax_new at the cursor, advances the cursor
 * (wrapping), and writes to *d_bias the bias Eq. 3 gives for the LARGEST entry of
 * the ring, minus `margin` -- the bias to quantise that tensor with at the next
 * step.  A ring that starts zero-filled ignores its unused entries; an all-zero
 * or non-finite maximum gives bias 0 and the status flag, as in fp8_scaling_bias.
 *   d_history  in/out: device float[len], 1 <= len <= 65536, owned by the caller
 *   d_cursor   in/out: device int32, index of the entry to overwrite next (0 at start)
 * len == 1 is fp8_scaling_bias on the newest amax. */
FP8_API fp8_status_t fp8_amax_history_bias(fp8_ctx *ctx, float *d_history, int32_t len, int32_t *d_cursor,
                                           const float *d_amax_new, fp8_format_t fmt, fp8_conv_t conv, int32_t margin,
                                           int32_t *d_bias, void *stream);

/* Bias log and bias mode (Appendix G plots, per tensor, the mode of the scaling bias over the data samples;
 * Appendix I its evolution per layer and step).  The log is a ring of records in device memory that the CALLER
 * owns and drains (a plain device-to-host copy of `capacity` records plus the head counter); nothing here
 * synchronises.
 *   fp8_bias_log_append  appends `count` records {step, first_tensor_id + i, d_amax[i], d_bias[i]}, i < count,
 *                        at the head of the ring (record n lives in slot n mod capacity; *d_head, a device
 *                        uint64 that starts at 0, counts every record ever appended).  d_amax / d_bias are
 *                        device arrays, e.g. the amax and bias words of all tensors of a step.  count <= capacity.
 *   fp8_bias_mode        over the records currently in the ring that carry `tensor_id` and a step in
 *                        [step_lo, step_hi]: *d_mode = their most frequent bias (the smaller value on a tie; 0
 *                        when there is none), *d_count = how often it occurs, *d_samples (may be NULL) = how
 *                        many records matched. */
typedef struct {
    int32_t step;
    int32_t tensor_id;
    float amax;
    int32_t bias;
} fp8_bias_record_t;
FP8_API fp8_status_t fp8_bias_log_append(fp8_ctx *ctx, fp8_bias_record_t *d_ring, int32_t capacity, uint64_t *d_head,
                                         int32_t step, int32_t first_tensor_id, const float *d_amax, const int32_t *d_bias,
                                         int32_t count, void *stream);
FP8_API fp8_status_t fp8_bias_mode(fp8_ctx *ctx, const fp8_bias_record_t *d_ring, int32_t capacity, const uint64_t *d_head,
                                   int32_t tensor_id, int32_t step_lo, int32_t step_hi, int32_t *d_mode, int32_t *d_count,
                                   int32_t *d_samples, void *stream);

/* The same integer rule on the host (no device work, no ctx). */
FP8_API fp8_status_t fp8_scaling_bias_host(float amax, fp8_format_t fmt, fp8_conv_t conv, int32_t margin, int32_t *bias);

/* Scale-and-cast (Eq. 1 then the cast of Section 2.1): code = RNE_fp8(x * 2^(bias + delta)),
 * saturating at the format's largest finite value; NaN stays NaN.
 *   x          [rows, cols], leading dimension ld, dtype x_dt (FP8_BF16, FP8_F16 or FP8_F32)
 *   d_bias     device int32, the paper-convention bias to apply.  Passing a
 *              constant chosen by the caller is the paper's FP8-CSCALE.
 *              NULL selects FP8-AMAX: amax and bias are computed here first
 *              (with `margin`) and written to d_amax_out / d_bias_out, both
 *              then required.
 *              Non-NULL together with non-NULL d_amax_out and d_bias_out is
 *              delayed scaling (the remedy Section 3 mentions for hardware
 *              where the second pass is too costly): the cast uses d_bias, and
 *              the same pass also writes this tensor's own amax and the bias
 *              Eq. 3 gives for it, for use at the next step.  d_bias_out may be
 *              the same word as d_bias.
 *   y          out [rows, cols] bytes, contiguous, or NULL
 *   y_t        out [cols, rows] bytes (the transposed copy, same codes), or NULL
 * At least one of y, y_t.  The vectorised paths need 16-byte aligned x, y, y_t,
 * ld % 8 == 0, and rows % 4 == 0 for y_t; other shapes take a slower guarded path. */
FP8_API fp8_status_t fp8_cast_e4(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                         const int32_t *d_bias, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                         int32_t *d_bias_out, uint8_t *y, uint8_t *y_t, void *stream);
/* Same for the gradient format E5 (Section 2.2). */
FP8_API fp8_status_t fp8_cast_e5(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                         const int32_t *d_bias, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                         int32_t *d_bias_out, uint8_t *y, uint8_t *y_t, void *stream);

/* FP8-AMAX in a single pass over the tensor when the bias can be guessed
 * (Section 3 names the problem -- just-in-time scaling costs a second round
 * trip to memory -- and the remedy of leaning on the amax history; Appendix I
 * shows how rarely the biases move).  *d_bias_inout holds a GUESS on entry,
 * typically what the previous step left there.  The tensor is cast with the
 * guess while its amax is taken in the same pass; the true bias is then
 * compared with the guess and, only if they differ, the cast is redone.  On
 * return d_amax_out, d_bias_inout and y are exactly what fp8_cast_e4 / _e5 with
 * d_bias = NULL would have written, whatever the guess was (any int32 is a valid
 * guess).  Cost: 3 bytes per element when the guess holds, 6 when it does not
 * (the two-launch path always moves 5).
 *   x   [rows, cols], dtype x_dt; the one-pass kernel needs ld == cols and
 *       16-byte aligned x and y, other tensors silently take the two-launch path
 *   y   out [rows, cols] bytes (row-major only)
 * Two launches are always made (the second returns at once when the guess held). */
FP8_API fp8_status_t fp8_cast_predicted(fp8_ctx *ctx, fp8_format_t fmt, const void *x, fp8_dtype_t x_dt, int64_t rows,
                                        int64_t cols, int64_t ld, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                                        int32_t *d_bias_inout, uint8_t *y, void *stream);

/* FP8-AMAX quantisation of several tensors in one call (Eq. 3, Eq. 1 and the casts of Sections 2.1 / 2.2,
 * per tensor; the grouping itself has no counterpart in the paper).  Every linear of a step quantises its
 * weight, and a step usually has several tensors ready at once (all weights after the optimiser update; in a
 * benchmark also the activations and gradients).  Launched one by one, kernels over tens of megabytes spend a
 * sizeable share of their time ramping up and draining; this call walks the chunks of all tensors with one
 * persistent grid per pass, two launches for the whole group.
 *   items      HOST array of `count` descriptors (read during the call, not retained); each tensor gets its own
 *              amax and bias, exactly as fp8_cast_e4 / fp8_cast_e5 with d_bias = NULL would give:
 *                x, x_dt, rows, cols, ld   the input tensor
 *                fmt, margin               target format and the margin subtracted from its Eq. 3 bias
 *                d_amax                    out, device float
 *                d_bias                    out, device int32; IN as well in the modes that start from a given bias
 *                y                         out [rows, cols] bytes, row-major
 *   mode       FP8_GROUP_AMAX_CAST: just in time -- one pass takes every amax and bias, a second casts (5 bytes
 *              moved per 16-bit element).
 *              FP8_GROUP_PREDICTED: one pass casts every tensor with the guess found in its d_bias (typically the
 *              value the previous step left there) while taking its amax; tensors whose guess turns out wrong
 *              are cast again by the second launch, the others are not touched again (3 bytes per element when
 *              all guesses hold; fp8_prediction_stats counts hits and misses).  Same results as
 *              FP8_GROUP_AMAX_CAST, whatever the guesses.
 *              FP8_GROUP_AMAX_ONLY: the first pass alone: d_amax and d_bias of every tensor (y may be NULL).
 *              FP8_GROUP_CAST_ONLY: the second pass alone, with the biases found in d_bias (chosen by the caller:
 *              FP8-CSCALE, or biases from an amax history); d_amax is not touched and may be NULL.
 * Tensors with ld == cols and 16-byte aligned x and y are grouped (up to FP8_GROUP_MAX of one input type per pair
 * of launches; more, or mixed types, are taken in several rounds); any other tensor in the list is handed to
 * fp8_amax / fp8_cast_e4 / _e5 / _predicted. */
#define FP8_GROUP_MAX 16
typedef struct {
    const void *x;
    fp8_dtype_t x_dt;
    int64_t rows, cols, ld;
    fp8_format_t fmt;
    int32_t margin;
    float *d_amax;
    int32_t *d_bias;
    uint8_t *y;
} fp8_group_item_t;
typedef enum { FP8_GROUP_AMAX_CAST = 0, FP8_GROUP_PREDICTED = 1, FP8_GROUP_AMAX_ONLY = 2, FP8_GROUP_CAST_ONLY = 3 } fp8_group_mode_t;
FP8_API fp8_status_t fp8_cast_group(fp8_ctx *ctx, const fp8_group_item_t *items, int32_t count, fp8_conv_t conv,
                                    fp8_group_mode_t mode, void *stream);

/* Synchronises `stream` and returns how many guesses of fp8_cast_predicted held / did not hold since the
 * context was created or the counters were last cleared. */
FP8_API fp8_status_t fp8_prediction_stats(fp8_ctx *ctx, void *stream, unsigned *hits, unsigned *misses, int clear);

/* Range statistics of a tensor under a given scaling bias, without casting it (for constant-bias sweeps as in
 * Section 4 / Appendix F, FP8-CSCALE: which biases keep a tensor inside the FP8 range).
 *   d_counts  out, four device uint64 (8-byte aligned), set by this call:
 *             [0] elements that would be clipped to the format's maximum (infinities included)
 *             [1] non-zero finite elements that would be flushed to zero
 *             [2] elements that would land in the format's subnormal range
 *             [3] non-zero finite elements of the tensor
 *   NaNs are not counted anywhere.  x may be strided (ld) and of any of the three input types. */
FP8_API fp8_status_t fp8_range_stats(fp8_ctx *ctx, fp8_format_t fmt, const void *x, fp8_dtype_t x_dt, int64_t rows,
                                     int64_t cols, int64_t ld, const int32_t *d_bias, fp8_conv_t conv,
                                     unsigned long long *d_counts, void *stream);

/* Post-training quantisation of one weight tensor (Section 3.1): amax -> bias
 * -> cast to E4, once.  w [N, K] (ld elements); outputs w8 [N, K] and/or
 * w8_t [K, N], d_bw, d_amax_w (both required). */
FP8_API fp8_status_t fp8_ptq_weights(fp8_ctx *ctx, const void *w, fp8_dtype_t w_dt, int64_t N, int64_t K, int64_t ld,
                             fp8_conv_t conv, uint8_t *w8, uint8_t *w8_t, int32_t *d_bw, float *d_amax_w,
                             void *stream);

/* Forward matmul with unscale (Fig. 3b, Eq. 2):
 *   Y[t, n] = (sum_k X8[t, k] * W8[n, k]) * 2^-(s_x + s_w) + bias_vec[n]
 * with s = bias + delta, FP32 accumulation on the tensor cores.
 *   x8 [T, K] E4 bytes, w8 [N, K] E4 bytes, both contiguous, 16-byte aligned, K % 16 == 0
 *   d_bx, d_bw  device int32 paper-convention biases of X and W
 *   bias_vec    NULL or [N] of dtype bias_dt (FP8_BF16 or FP8_F32), added after the unscale
 *   y           out [T, N] contiguous, dtype y_dt (FP8_BF16 or FP8_F32)
 *   d_amax_y    NULL, or out: amax of the rounded output (set by this call)
 */
FP8_API fp8_status_t fp8_linear_fwd(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                            const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y,
                            fp8_dtype_t y_dt, float *d_amax_y, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                            void *stream);

/* The forward matmul of inference on weights quantised once (Section 3.1: post-training quantisation, the weights'
 * scaling bias and bytes are fixed, the activations are quantised per call).  Arguments, result and errors are
 * those of fp8_linear_fwd, bit for bit.  One more condition on the caller, and what it buys: the bytes of w8 must
 * have been final before the launch that precedes this call on `stream` began (true of weights produced once by
 * fp8_ptq_weights and then left alone; NOT true when w8 comes out of a cast enqueued just before).  With at most 128
 * rows the matmul then starts streaming weight tiles while that launch (typically the cast of the few activation
 * rows) is still running, instead of after it; x8, d_bx, d_bw and bias_vec are still read only once it has
 * completed.  With more rows the call is fp8_linear_fwd. */
FP8_API fp8_status_t fp8_linear_infer(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                              const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y,
                              fp8_dtype_t y_dt, float *d_amax_y, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                              void *stream);

/* Inference on a few rows in one launch (Section 3.1: the activation is quantised per call, the weights once):
 * FP8-AMAX of the activation (Eq. 3, then Eq. 1 and the E4 cast) followed by the forward matmul.  Results are those
 * of fp8_cast_e4 (d_bias = NULL, FP8-AMAX) followed by fp8_linear_infer, bit for bit: d_amax_x, d_bx and the bytes
 * x8 [T, K] are outputs of this call (all three required; x8 16-byte aligned), y as in fp8_linear_fwd.
 *   x    [T, K] contiguous, dtype x_dt
 * With an activation of at most 64 KB (one row of 28672 elements, four rows of 8192), bf16 and 16-byte aligned, one
 * kernel does both steps: every CTA takes the amax of the whole of x, derives the bias and casts x for itself (all
 * write the same bytes to x8), then multiplies, while its weight tiles have been streaming since the kernel began.
 * Any other case runs the two calls.  The condition of fp8_linear_infer on w8 applies. */
FP8_API fp8_status_t fp8_linear_infer_cast(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int32_t margin, float *d_amax_x,
                                   int32_t *d_bx, uint8_t *x8, const uint8_t *w8, const int32_t *d_bw,
                                   const void *bias_vec, fp8_dtype_t bias_dt, void *y, fp8_dtype_t y_dt,
                                   float *d_amax_y, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream);

/* Several independent matmuls in one launch (the paper has no counterpart; Section 2.2 is where they come from: the
 * input-gradient and weight-gradient matmuls of a layer share dY8 and do not depend on each other, nor do the
 * matmuls of different layers whose operands are ready).  Each item is one fp8_linear_fwd, fp8_linear_dgrad or
 * fp8_linear_wgrad call on row-major operands, with that call's meaning, checks and results (the FP32 sums may be
 * taken in another order than the member's own launch would take them: same bars, not always the same last bit):
 *   FP8_MATMUL_FWD    a8 = x8 [T, K] (E4),  b8 = w8 [N, K] (E4), out = Y [T, N]; bias_vec / bias_dt as in fp8_linear_fwd
 *   FP8_MATMUL_DGRAD  a8 = dy8 [T, N] (E5), b8 = w8 [N, K] (E4), out = dX [T, K]   (fp8_linear_dgrad with w8_t = NULL)
 *   FP8_MATMUL_WGRAD  a8 = dy8 [T, N] (E5), b8 = x8 [T, K] (E4), out = dW [N, K]   (fp8_linear_wgrad with both
 *                     transposed copies NULL); d_amax_out must be NULL
 *   d_ba, d_bb        device int32 biases of a8 and b8;  out_dt FP8_BF16 or FP8_F32;  d_amax_out NULL or the amax of out
 * No item may read what another item of the same call writes.  `items` is a HOST array, read during the call only.
 * With at most 16 items, all of more than 128 output rows, one persistent kernel walks the output tiles of all
 * items in one sequence (shortest contractions first), so the launch pays one ramp and one drain and the last wave
 * of one matmul is filled with the first tiles of the next; any other group runs as its members' own calls, in
 * order.  Argument errors of any member of a one-launch group are returned before the launch (the d_amax_out words
 * of members listed before the faulty one may already have been cleared). */
typedef enum { FP8_MATMUL_FWD = 0, FP8_MATMUL_DGRAD = 1, FP8_MATMUL_WGRAD = 2 } fp8_matmul_kind_t;
typedef struct {
    int32_t kind;            /* fp8_matmul_kind_t */
    int32_t bias_dt;         /* fp8_dtype_t of bias_vec (FWD) */
    const uint8_t *a8;
    const int32_t *d_ba;
    const uint8_t *b8;
    const int32_t *d_bb;
    const void *bias_vec;    /* FWD: NULL or [N]; otherwise NULL */
    void *out;
    float *d_amax_out;
    int32_t out_dt;          /* fp8_dtype_t */
    int32_t reserved;        /* 0 */
    int64_t T, K, N;         /* of the layer: tokens, in-features, out-features */
} fp8_matmul_item_t;
FP8_API fp8_status_t fp8_linear_group(fp8_ctx *ctx, const fp8_matmul_item_t *items, int32_t count, fp8_conv_t conv,
                              void *stream);

/* Forward matmul with the activation fused into the epilogue (the paper has no
 * counterpart; it answers Section 3's warning that computing a scale just in
 * time costs a second pass over memory: the next layer's input leaves this
 * kernel together with its amax, so that layer needs no amax pass).
 *   y_pre  NULL, or out [T, N] bf16: the rounded pre-activation
 *          (unscale, + bias_vec), what the backward pass of the activation needs
 *   y_act  out [T, N] bf16: act(y_pre), evaluated in FP32 on the bf16-rounded
 *          pre-activation, i.e. on exactly what y_pre holds
 *   act    FP8_ACT_GELU: x/2 * (1 + erf(x / sqrt 2)), through a fitted form of the
 *          normal distribution function whose bf16 result is within one bf16 ulp of
 *          the correctly rounded value for every finite bf16 input (GELU' in the
 *          backward twin: within 1.2e-4 relative before rounding); a non-finite
 *          pre-activation gives a non-finite output
 *   d_amax_act  NULL or out: amax of y_act; fp8_scaling_bias + fp8_cast_e4 with
 *          that bias then quantise y_act in a single pass
 *          FP8_ACT_SWIGLU: the gated unit of the Llama MLP, z = SiLU(gate) * up with
 *          SiLU(a) = a / (1 + exp(-a)).  The caller stores the gate and the up
 *          projection as ONE weight w8[N = 2F, K] whose rows come in blocks of 64:
 *          32 gate rows (features 32b .. 32b+31) followed by the 32 up rows of the
 *          same features; y_pre [T, 2F] has that column layout, y_act is [T, F].
 *          Both factors are the bf16-rounded pre-activations; the bf16 result is
 *          within one bf16 ulp of the correctly rounded product.  Needs N % 64 == 0.
 * Needs 16-byte aligned y_pre / y_act and N % 8 == 0, besides fp8_linear_fwd's rules. */
typedef enum { FP8_ACT_NONE = 0, FP8_ACT_GELU = 1, FP8_ACT_SWIGLU = 2 } fp8_act_t;
FP8_API fp8_status_t fp8_linear_fwd_act(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                                        const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y_pre,
                                        void *y_act, fp8_act_t act, float *d_amax_act, int64_t T, int64_t K, int64_t N,
                                        fp8_conv_t conv, void *stream);

/* Input-gradient matmul (Section 2.2): dX[t, k] = (sum_n dY8[t, n] * W8[n, k]) * 2^-(s_g + s_w).
 *   dy8  [T, N] E5 bytes;  N % 16 == 0
 *   w8   [N, K] E4 bytes or NULL;  w8_t [K, N] E4 bytes or NULL.  At least one.
 *        With w8_t (as written by the cast's y_t) the contraction runs over
 *        contiguous bytes; with w8 alone the tensor core reads W8 with its K
 *        index contiguous and the contraction strided (needs K % 16 == 0), so
 *        no transposed copy is required.  w8_t is used when both are given.
 *   dx   out [T, K], dtype dx_dt;  d_amax_dx NULL or out. */
FP8_API fp8_status_t fp8_linear_dgrad(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                              const uint8_t *w8_t, const int32_t *d_bw, void *dx, fp8_dtype_t dx_dt,
                              float *d_amax_dx, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream);

/* Input-gradient matmul with the activation's backward fused into the epilogue (no counterpart in the paper;
 * the backward twin of fp8_linear_fwd_act).  With y_pre [T, K] the bf16 pre-activation that produced this
 * layer's input (X = act(y_pre)):
 *   dx      NULL, or out [T, K] bf16: the rounded input gradient dX
 *   dx_act  out [T, K] bf16: bf16(dX) * act'(y_pre) in FP32, rounded -- the output gradient of the layer below
 *   d_amax_act  NULL or out: its amax, so that the layer below quantises it in a single pass
 * With FP8_ACT_SWIGLU the matmul's output dX[T, K] is the gradient dz of the gated
 * unit's output; y_pre is the stored [T, 2K] pre-activation in the block layout of
 * fp8_linear_fwd_act, and dx_act [T, 2K] receives, in the same layout,
 *   d_gate = bf16(dz) * up * SiLU'(gate),  d_up = bf16(dz) * SiLU(gate),
 * SiLU'(a) = s + a s (1 - s), s = 1 / (1 + exp(-a)); d_amax_act covers both.  Needs K % 32 == 0.
 * Operand rules as fp8_linear_dgrad; y_pre, dx, dx_act 16-byte aligned, K % 8 == 0. */
FP8_API fp8_status_t fp8_linear_dgrad_act(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                                          const uint8_t *w8_t, const int32_t *d_bw, const void *y_pre, void *dx,
                                          void *dx_act, fp8_act_t act, float *d_amax_act, int64_t T, int64_t K,
                                          int64_t N, fp8_conv_t conv, void *stream);

/* Matmuls whose result leaves already quantised, for a bias known before the
 * launch (no counterpart in the paper beyond Section 3's remark that a scale may
 * rely on the history of amax instead of a second pass over memory: here the
 * consumer's FP8 bytes are written by the producer's epilogue, and the amax that
 * feeds the history comes out of the same launch).  The 16-bit tensor z the
 * bytes are made from is
 *   fp8_linear_fwd_q:   z = bf16(Y) for FP8_ACT_NONE, z = bf16(GELU(bf16(Y))) for FP8_ACT_GELU,
 *                       Y as in fp8_linear_fwd;  z8 = E4 bytes of z under bias *d_bz
 *   fp8_linear_dgrad_q: z = bf16(dX) for FP8_ACT_NONE, z = bf16(bf16(dX) * GELU'(y_pre)) for FP8_ACT_GELU,
 *                       dX as in fp8_linear_dgrad;  g8 = E5 bytes of z under bias *d_bq
 *   FP8_ACT_SWIGLU:     as in fp8_linear_fwd_act / fp8_linear_dgrad_act: forward z and z8 are [T, N/2],
 *                       backward y_pre, g and g8 are [T, 2K] (N % 64 == 0, K % 32 == 0)
 * and the bytes are exactly what fp8_cast_e4 / fp8_cast_e5 with that bias give on
 * the stored z (FP8_FLAG_SATURATED is raised likewise when a value clips).
 *   y_pre (fwd)   NULL, or out [T, N] bf16 pre-activation; must be NULL with FP8_ACT_NONE
 *   y_pre (dgrad) in [T, K] bf16 pre-activation, required with FP8_ACT_GELU, NULL otherwise
 *   dx            NULL, or out [T, K] bf16 rounded dX; must be NULL with FP8_ACT_NONE
 *   z / g         NULL, or out bf16: the tensor the bytes are made from
 *   z8 / g8       out bytes, [T, N] / [T, K], 16-byte aligned; N % 16 == 0 (fwd), K % 16 == 0 (dgrad)
 *   d_bz / d_bq   in: device int32, paper-convention bias to quantise with (the caller's prediction)
 *   d_amax_z / d_amax_g  NULL or out: amax of z, from which the caller updates its prediction
 * Other operands as in fp8_linear_fwd / fp8_linear_dgrad; 16-bit outputs 16-byte aligned. */
FP8_API fp8_status_t fp8_linear_fwd_q(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                                      const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, fp8_act_t act,
                                      void *y_pre, void *z, uint8_t *z8, const int32_t *d_bz, float *d_amax_z,
                                      int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream);
FP8_API fp8_status_t fp8_linear_dgrad_q(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                                        const uint8_t *w8_t, const int32_t *d_bw, fp8_act_t act, const void *y_pre,
                                        void *dx, void *g, uint8_t *g8, const int32_t *d_bq, float *d_amax_g,
                                        int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream);

/* Weight-gradient matmul (Section 2.2): dW[n, k] = (sum_t dY8[t, n] * X8[t, k]) * 2^-(s_g + s_x).
 *   dy8 [T, N] / dy8_t [N, T] E5 bytes, x8 [T, K] / x8_t [K, T] E4 bytes.
 *   Each operand in either layout (the transposed copy wins when both are
 *   given): a transposed copy needs T % 16 == 0; dy8 needs N % 16 == 0 and x8
 *   needs K % 16 == 0.  No transposed copy is required.
 *   dw  out [N, K], dtype dw_dt. */
FP8_API fp8_status_t fp8_linear_wgrad(fp8_ctx *ctx, const uint8_t *dy8, const uint8_t *dy8_t, const int32_t *d_bg,
                              const uint8_t *x8, const uint8_t *x8_t, const int32_t *d_bx, void *dw,
                              fp8_dtype_t dw_dt, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream);

/* The paper's own accumulation regime, emulated (Fig. 3b: FP8 inputs, partial results accumulated in FP16, FP16
 * output; Section 2.4: why loss scaling returns with FP16 accumulation; Section 3.2: the margin that keeps the two
 * backward matmuls from overflowing FP16).  The paper does not say how many products its hardware adds before it
 * rounds; here the granularity is the argument `chunk`: the products of `chunk` consecutive contraction indices
 * (a multiple of 128) are accumulated on the tensor cores in FP32 -- exact to 2^-21 of their absolute sum -- each such
 * partial sum is added to a running FP16 accumulator with one rounding to FP16 (beyond 65504 it becomes infinite and
 * stays so), and the FP16 result is unscaled in FP16 (Eq. 2 applied to the FP16 output: one more rounding only where
 * the result leaves FP16's normal range).  For studying margins and loss scales, not for speed (an eighth of the plain
 * matmul's rate at chunk = 128, two thirds at chunk = 2048).  Operands in their forward layouts:
 *   FP8_MM_FWD    a8 = X8[T,K] (E4), b8 = W8[N,K] (E4)  ->  out = Y[T,N]
 *   FP8_MM_DGRAD  a8 = dY8[T,N] (E5), b8 = W8[N,K] (E4)  ->  out = dX[T,K]
 *   FP8_MM_WGRAD  a8 = dY8[T,N] (E5), b8 = X8[T,K] (E4)  ->  out = dW[N,K]
 *   d_ba, d_bb    device int32 paper-convention biases of a8 and b8
 *   out           contiguous, 16-byte aligned, dtype FP8_F16 (IEEE half) or FP8_F32 (exactly the FP16 values)
 * K % 16 == 0, N % 16 == 0, and the output's row length a multiple of 8. */
typedef enum { FP8_MM_FWD = 0, FP8_MM_DGRAD = 1, FP8_MM_WGRAD = 2 } fp8_matmul_t;
FP8_API fp8_status_t fp8_linear_f16acc(fp8_ctx *ctx, fp8_matmul_t kind, const uint8_t *a8, const int32_t *d_ba,
                                       const uint8_t *b8, const int32_t *d_bb, void *out, fp8_dtype_t out_dt, int32_t chunk,
                                       int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FP8LIN_H */
