/*
 * fp8_harness.h -- element-wise kernels of the dynamic-scaling stress workload (a stack of FP8 linears with GELU
 * between them, a mean-squared-error loss and plain SGD).  None of this is the paper's method: the paper quantises
 * the linears of a decoder and leaves everything else in higher precision.  These calls are that "everything
 * else" for the stress stack, as CUDA kernels in the same library so that a step of the stack launches no
 * framework kernels of its own.
 *
 * Conventions: device pointers owned by the caller, contiguous tensors of `n` elements, bf16 unless stated,
 * FP32 arithmetic with one rounding to bf16 at the end (round to nearest even), asynchronous on `stream`
 * (a cudaStream_t passed as void*).  Pointers must be 2-byte (bf16) / 4-byte (fp32) aligned; any n > 0.
 * Errors (NULL, n <= 0) are returned before anything is launched.
 */
#ifndef FP8_HARNESS_H
#define FP8_HARNESS_H

#include "fp8lin.h"

#ifdef __cplusplus
extern "C" {
#endif

/* y = bf16( x * Phi(x) ), Phi(x) = erfc(-x / sqrt 2) / 2: GELU of the bf16 value in FP32 (the complementary error
 * function keeps the negative tail's relative accuracy). */
FP8_API fp8_status_t fp8h_gelu(const void *x, void *y, int64_t n, void *stream);

/* out = bf16( g * GELU'(pre) ),  GELU'(z) = Phi(z) + z * phi(z): the gradient through a GELU whose input was `pre`. */
FP8_API fp8_status_t fp8h_gelu_backward(const void *g, const void *pre, void *out, int64_t n, void *stream);

/* g = bf16( (y - target) * scale ): gradient of a mean-squared-error loss (scale = 2 / number of elements). */
FP8_API fp8_status_t fp8h_mse_grad(const void *y, const void *target, float scale, void *g, int64_t n, void *stream);

/* Plain SGD on FP32 master weights with the 16-bit copy the next forward pass quantises:
 *   w32 <- w32 - lr * dw   (one fused multiply-add per element),   w16 = bf16(w32).
 * w32 [n] fp32 in / out, dw [n] bf16, w16 [n] bf16 out. */
FP8_API fp8_status_t fp8h_sgd(float *w32, const void *dw, float lr, void *w16, int64_t n, void *stream);

#ifdef __cplusplus
}
#endif
#endif
