// amax (Eq. 3, first line) and the integer scaling bias (Eq. 3, second line).
//
// amax is a selection, not arithmetic: on bf16 bit patterns |x| orders like the
// unsigned integer (bits & 0x7FFF), with NaN > inf > finite.  The kernel keeps
// two 16-bit lanes per register (one packed max per 32-bit word), reduces by
// warp shuffle, then per block, then across the grid through one atomicMax per
// block on a context-owned slot; the last block to arrive publishes the result
// (and, when asked, the bias) and leaves the slot zeroed for the next call.
// HBM-bound: 2 bytes read per element, nothing written.
#include "fp8lin_internal.cuh"

namespace fp8lin {

constexpr int kAmaxThreads = 256;
constexpr int kAmaxUnroll = 4;  // 16-byte loads in flight per thread

struct AmaxOut {
    unsigned *slot;      // {running max, arrival counter}
    float *d_amax;
    int32_t *d_bias;     // may be NULL
    unsigned *d_status;
    int fmt, conv, margin;
};

__device__ __forceinline__ uint32_t packed_abs_max(uint32_t acc, uint32_t w)
{
    return __vmaxu2(acc, w & 0x7FFF7FFFu);
}

// Block-level reduction of a packed running max, then the grid-level step.
__device__ __forceinline__ void amax_finish(uint32_t packed, const AmaxOut &o)
{
    __shared__ uint32_t warp_max[kAmaxThreads / 32];
    uint32_t m = max(packed & 0xFFFFu, packed >> 16);
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 1; i < kAmaxThreads / 32; ++i) m = max(m, warp_max[i]);
        atomicMax(&o.slot[0], m);
        __threadfence();
        unsigned arrived = atomicAdd(&o.slot[1], 1u) + 1u;
        if (arrived == gridDim.x) {
            __threadfence();
            uint32_t total = atomicExch(&o.slot[0], 0u);
            o.slot[1] = 0u;
            uint32_t fbits = total << 16;  // bf16 -> float bit pattern
            *o.d_amax = __uint_as_float(fbits);
            unsigned flags = 0;
            int b = bias_from_amax_bits(fbits, o.fmt, o.conv, o.margin, &flags);
            if (o.d_bias) {
                *o.d_bias = b;
                if (flags) atomicOr(o.d_status, flags);
            }
        }
    }
}

// Contiguous tensor seen as nvec 16-byte vectors plus a scalar tail.
__global__ void __launch_bounds__(kAmaxThreads) amax_flat_kernel(const uint4 *__restrict__ x, int64_t nvec,
                                                                 const uint16_t *__restrict__ tail, int ntail,
                                                                 AmaxOut o)
{
    uint32_t acc = 0;
    const int64_t chunk = (int64_t)kAmaxThreads * kAmaxUnroll;
    for (int64_t base = (int64_t)blockIdx.x * chunk; base < nvec; base += (int64_t)gridDim.x * chunk) {
        uint4 v[kAmaxUnroll];
#pragma unroll
        for (int j = 0; j < kAmaxUnroll; ++j) {
            int64_t i = base + threadIdx.x + (int64_t)j * kAmaxThreads;
            v[j] = (i < nvec) ? __ldg(x + i) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kAmaxUnroll; ++j) {
            acc = packed_abs_max(acc, v[j].x);
            acc = packed_abs_max(acc, v[j].y);
            acc = packed_abs_max(acc, v[j].z);
            acc = packed_abs_max(acc, v[j].w);
        }
    }
    if (blockIdx.x == 0 && (int)threadIdx.x < ntail) acc = packed_abs_max(acc, (uint32_t)tail[threadIdx.x]);
    amax_finish(acc, o);
}

// General [rows, cols] with leading dimension ld; vec != 0 promises 16-byte
// aligned rows (x aligned, ld % 8 == 0).
__global__ void __launch_bounds__(kAmaxThreads) amax_rows_kernel(const uint16_t *__restrict__ x, int64_t rows,
                                                                 int64_t cols, int64_t ld, int vec, AmaxOut o)
{
    uint32_t acc = 0;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const uint16_t *row = x + r * ld;
        int64_t done = 0;
        if (vec) {
            int64_t nv = cols / 8;
            const uint4 *rv = reinterpret_cast<const uint4 *>(row);
            for (int64_t i = threadIdx.x; i < nv; i += kAmaxThreads) {
                uint4 v = __ldg(rv + i);
                acc = packed_abs_max(acc, v.x);
                acc = packed_abs_max(acc, v.y);
                acc = packed_abs_max(acc, v.z);
                acc = packed_abs_max(acc, v.w);
            }
            done = nv * 8;
        }
        for (int64_t c = done + threadIdx.x; c < cols; c += kAmaxThreads) acc = packed_abs_max(acc, (uint32_t)row[c]);
    }
    amax_finish(acc, o);
}

__global__ void scaling_bias_kernel(const float *__restrict__ d_amax, int fmt, int conv, int margin,
                                    int32_t *__restrict__ d_bias, unsigned *d_status)
{
    unsigned flags = 0;
    *d_bias = bias_from_amax_bits(__float_as_uint(*d_amax), fmt, conv, margin, &flags);
    if (flags) atomicOr(d_status, flags);
}

cudaError_t launch_amax_bias(fp8_ctx *ctx, const void *x, int64_t rows, int64_t cols, int64_t ld, float *d_amax,
                             int32_t *d_bias, int fmt, int conv, int margin, cudaStream_t stream)
{
    AmaxOut o{take_slot(ctx), d_amax, d_bias, ctx->d_status, fmt, conv, margin};
    const bool aligned = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    const int max_blocks = ctx->sm_count * 8;
    if (ld == cols && aligned) {
        int64_t n = rows * cols;
        int64_t nvec = n / 8;
        int ntail = (int)(n - nvec * 8);
        int64_t chunk = (int64_t)kAmaxThreads * kAmaxUnroll;
        int64_t want = (nvec + chunk - 1) / chunk;
        int blocks = (int)(want < 1 ? 1 : (want > max_blocks ? max_blocks : want));
        amax_flat_kernel<<<blocks, kAmaxThreads, 0, stream>>>(reinterpret_cast<const uint4 *>(x), nvec,
                                                             reinterpret_cast<const uint16_t *>(x) + nvec * 8, ntail,
                                                             o);
    } else {
        int vec = (aligned && (ld % 8) == 0) ? 1 : 0;
        int blocks = (int)(rows > max_blocks ? max_blocks : rows);
        amax_rows_kernel<<<blocks, kAmaxThreads, 0, stream>>>(reinterpret_cast<const uint16_t *>(x), rows, cols, ld,
                                                             vec, o);
    }
    return cudaGetLastError();
}

}  // namespace fp8lin

extern "C" {

fp8_status_t fp8_amax(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                      float *d_amax, void *stream)
{
    if (!ctx || !x || !d_amax) return FP8_ERR_NULL;
    if ((int)x_dt < 0 || (int)x_dt > 2) return FP8_ERR_DTYPE;
    if (x_dt != FP8_BF16) return FP8_ERR_UNSUPPORTED;
    if (rows <= 0 || cols <= 0 || ld < cols) return FP8_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(x) & 1u) return FP8_ERR_ALIGN;
    cudaError_t e = fp8lin::launch_amax_bias(ctx, x, rows, cols, ld, d_amax, nullptr, 0, 0, 0, (cudaStream_t)stream);
    return e == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_scaling_bias(fp8_ctx *ctx, const float *d_amax, fp8_format_t fmt, fp8_conv_t conv, int32_t margin,
                              int32_t *d_bias, void *stream)
{
    if (!ctx || !d_amax || !d_bias) return FP8_ERR_NULL;
    if ((int)fmt < 0 || (int)fmt > 1 || (int)conv < 0 || (int)conv > 1) return FP8_ERR_DTYPE;
    fp8lin::scaling_bias_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(d_amax, (int)fmt, (int)conv, margin, d_bias,
                                                                  ctx->d_status);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

}  // extern "C"
