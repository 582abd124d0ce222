// Element-wise kernels of the stress stack (GELU, its derivative, the loss gradient, SGD): harness, not method.
// Memory-bound, one pass each, 16-byte vectors where the pointers allow, scalar otherwise.
#include "fp8_harness.h"
#include "fp8lin_internal.cuh"

namespace fp8lin {

__device__ __forceinline__ float bf16_to_f32(uint16_t h) { return __uint_as_float((uint32_t)h << 16); }
__device__ __forceinline__ uint16_t f32_to_bf16(float v)
{
    uint32_t w;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(0.0f), "f"(v));
    return (uint16_t)(w & 0xFFFFu);
}

// every product and sum is rounded to FP32 on its own (no contraction into fused multiply-adds): the result does
// not depend on how a compiler pairs the operations
// Phi(z) = erfc(-z / sqrt 2) / 2 rather than (1 + erf(z / sqrt 2)) / 2: the latter cancels in the negative tail
__device__ __forceinline__ float normal_cdf_f32(float z) { return __fmul_rn(0.5f, erfcf(__fmul_rn(z, -0.70710678118654752440f))); }
__device__ __forceinline__ float gelu_f32(float z) { return __fmul_rn(z, normal_cdf_f32(z)); }
__device__ __forceinline__ float gelu_grad_f32_exact(float z)
{
    const float pdf = __fmul_rn(expf(__fmul_rn(-0.5f, __fmul_rn(z, z))), 0.39894228040143267794f);
    return __fadd_rn(normal_cdf_f32(z), __fmul_rn(z, pdf));
}

enum { kGelu = 0, kGeluBackward = 1, kMseGrad = 2 };

// out[i] = f(a[i], b[i]); grid-stride over elements, eight per thread per trip when everything is 16-byte aligned
template <int OP>
__global__ void __launch_bounds__(256) harness_map_kernel(const uint16_t *__restrict__ a, const uint16_t *__restrict__ b,
                                                          uint16_t *__restrict__ out, float scale, int64_t n, int vec)
{
    auto f = [&](uint16_t x, uint16_t y) -> uint16_t {
        if (OP == kGelu) return f32_to_bf16(gelu_f32(bf16_to_f32(x)));
        if (OP == kGeluBackward) return f32_to_bf16(__fmul_rn(bf16_to_f32(x), gelu_grad_f32_exact(bf16_to_f32(y))));
        return f32_to_bf16(__fmul_rn(__fsub_rn(bf16_to_f32(x), bf16_to_f32(y)), scale));
    };
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    if (vec) {
        const int64_t nv = n / 8;
        for (int64_t i = tid; i < nv; i += stride) {
            const uint4 va = __ldcs(reinterpret_cast<const uint4 *>(a) + i);
            const uint4 vb = OP == kGelu ? va : __ldcs(reinterpret_cast<const uint4 *>(b) + i);
            const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
            uint32_t wo[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                wo[j] = (uint32_t)f((uint16_t)(wa[j] & 0xFFFFu), (uint16_t)(wb[j] & 0xFFFFu)) |
                        ((uint32_t)f((uint16_t)(wa[j] >> 16), (uint16_t)(wb[j] >> 16)) << 16);
            __stcs(reinterpret_cast<uint4 *>(out) + i, make_uint4(wo[0], wo[1], wo[2], wo[3]));
        }
        for (int64_t i = nv * 8 + tid; i < n; i += stride) out[i] = f(a[i], OP == kGelu ? a[i] : b[i]);
    } else {
        for (int64_t i = tid; i < n; i += stride) out[i] = f(a[i], OP == kGelu ? a[i] : b[i]);
    }
}

__global__ void __launch_bounds__(256) harness_sgd_kernel(float *__restrict__ w32, const uint16_t *__restrict__ dw, float neg_lr,
                                                          uint16_t *__restrict__ w16, int64_t n)
{
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = tid; i < n; i += stride) {
        const float w = __fmaf_rn(neg_lr, bf16_to_f32(dw[i]), w32[i]);
        w32[i] = w;
        w16[i] = f32_to_bf16(w);
    }
}

static bool aligned16p(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static unsigned grid_for(int64_t work)
{
    int64_t blocks = (work + 255) / 256;
    const int64_t cap = 148 * 8;
    return (unsigned)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

template <int OP>
static fp8_status_t launch_map(const void *a, const void *b, void *out, float scale, int64_t n, void *stream)
{
    if (!a || !out || (OP != kGelu && !b)) return FP8_ERR_NULL;
    if (n <= 0) return FP8_ERR_SHAPE;
    const int vec = aligned16p(a) && aligned16p(out) && (OP == kGelu || aligned16p(b)) ? 1 : 0;
    count_launch();
    harness_map_kernel<OP><<<grid_for(vec ? n / 8 + 1 : n), 256, 0, (cudaStream_t)stream>>>(
        static_cast<const uint16_t *>(a), static_cast<const uint16_t *>(b), static_cast<uint16_t *>(out), scale, n, vec);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

}  // namespace fp8lin

extern "C" {

fp8_status_t fp8h_gelu(const void *x, void *y, int64_t n, void *stream)
{
    return fp8lin::launch_map<fp8lin::kGelu>(x, nullptr, y, 0.0f, n, stream);
}

fp8_status_t fp8h_gelu_backward(const void *g, const void *pre, void *out, int64_t n, void *stream)
{
    return fp8lin::launch_map<fp8lin::kGeluBackward>(g, pre, out, 0.0f, n, stream);
}

fp8_status_t fp8h_mse_grad(const void *y, const void *target, float scale, void *g, int64_t n, void *stream)
{
    return fp8lin::launch_map<fp8lin::kMseGrad>(y, target, g, scale, n, stream);
}

fp8_status_t fp8h_sgd(float *w32, const void *dw, float lr, void *w16, int64_t n, void *stream)
{
    if (!w32 || !dw || !w16) return FP8_ERR_NULL;
    if (n <= 0) return FP8_ERR_SHAPE;
    fp8lin::count_launch();
    fp8lin::harness_sgd_kernel<<<fp8lin::grid_for(n), 256, 0, (cudaStream_t)stream>>>(
        w32, static_cast<const uint16_t *>(dw), -lr, static_cast<uint16_t *>(w16), n);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

}  // extern "C"
