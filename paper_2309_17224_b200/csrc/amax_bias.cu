// amax (Eq. 3, first line) and the integer scaling bias (Eq. 3, second line).
//
// amax is a selection, not arithmetic: on the bit patterns of bf16, fp16 and
// fp32 alike |x| orders like the unsigned integer with the sign bit cleared,
// with NaN > inf > finite.  For the 16-bit types the kernels keep two lanes
// per register (one packed max per 32-bit word); they reduce by
// warp shuffle, then per block, then across the grid through one atomicMax per
// block on a context-owned slot; the last block to arrive publishes the result
// (and, when asked, the bias) and leaves the slot zeroed for the next call.
// HBM-bound: 2 bytes read per element, nothing written.  Contiguous tensors take
// the streaming kernel of group.cu; this file holds the strided form.
#include "fp8lin_internal.cuh"

namespace fp8lin {

constexpr int kAmaxThreads = 256;

struct AmaxOut {
    unsigned *slot;      // {running max, arrival counter}
    float *d_amax;
    int32_t *d_bias;     // may be NULL
    unsigned *d_status;
    int fmt, conv, margin;
};

// |x| orders like an unsigned integer on the bit pattern with the sign cleared (NaN > inf > finite) for all
// three input types.  16-bit types keep two lanes per word; fp32 one.
template <int DT>
__device__ __forceinline__ uint32_t fold_word(uint32_t acc, uint32_t w)
{
    return DT == FP8_F32 ? max(acc, w & 0x7FFFFFFFu) : __vmaxu2(acc, w & 0x7FFF7FFFu);
}
template <int DT>
__device__ __forceinline__ uint32_t fold_elem(uint32_t acc, const void *x, int64_t i)
{
    if (DT == FP8_F32) return max(acc, reinterpret_cast<const uint32_t *>(x)[i] & 0x7FFFFFFFu);
    return __vmaxu2(acc, (uint32_t)reinterpret_cast<const uint16_t *>(x)[i] & 0x7FFFu);
}
template <int DT>
__device__ __forceinline__ uint32_t lane_key(uint32_t acc)
{
    return DT == FP8_F32 ? acc : max(acc & 0xFFFFu, acc >> 16);
}
// the winning bit pattern as float bits
template <int DT>
__device__ __forceinline__ uint32_t key_to_float_bits(uint32_t key)
{
    if (DT == FP8_F32) return key;
    if (DT == FP8_BF16) return key << 16;
    float f;
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"((uint16_t)key));
    return __float_as_uint(f);
}

// Block-level reduction of a running max, then the grid-level step.
template <int DT>
__device__ __forceinline__ void amax_finish(uint32_t acc, const AmaxOut &o)
{
    __shared__ uint32_t warp_max[kAmaxThreads / 32];
    uint32_t m = lane_key<DT>(acc);
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
            uint32_t fbits = key_to_float_bits<DT>(total);
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

// General [rows, cols] with leading dimension ld; vec != 0 promises 16-byte aligned rows.
template <int DT>
__global__ void __launch_bounds__(kAmaxThreads) amax_rows_kernel(const void *__restrict__ x, int64_t rows,
                                                                 int64_t cols, int64_t ld, int vec, AmaxOut o)
{
    constexpr int kPerVec = DT == FP8_F32 ? 4 : 8;
    constexpr int kB = DT == FP8_F32 ? 4 : 2;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    uint32_t acc = 0;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        int64_t done = 0;
        if (vec) {
            int64_t nv = cols / kPerVec;
            const uint4 *rv = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint8_t *>(x) + r * ld * kB);
            for (int64_t i = threadIdx.x; i < nv; i += kAmaxThreads) {
                uint4 v = __ldg(rv + i);
                acc = fold_word<DT>(acc, v.x);
                acc = fold_word<DT>(acc, v.y);
                acc = fold_word<DT>(acc, v.z);
                acc = fold_word<DT>(acc, v.w);
            }
            done = nv * kPerVec;
        }
        for (int64_t c = done + threadIdx.x; c < cols; c += kAmaxThreads) acc = fold_elem<DT>(acc, x, r * ld + c);
    }
    amax_finish<DT>(acc, o);
}

__global__ void scaling_bias_kernel(const float *__restrict__ d_amax, int fmt, int conv, int margin,
                                    int32_t *__restrict__ d_bias, unsigned *d_status)
{
    unsigned flags = 0;
    *d_bias = bias_from_amax_bits(__float_as_uint(*d_amax), fmt, conv, margin, &flags);
    if (flags) atomicOr(d_status, flags);
}

// One warp: push the newest amax into the ring, take the largest entry (|x| orders like its bit pattern; NaN and
// inf sort above every finite value and end up flagged by the bias rule), derive the bias.
__global__ void amax_history_kernel(float *__restrict__ d_history, int len, int32_t *__restrict__ d_cursor,
                                    const float *__restrict__ d_amax_new, int fmt, int conv, int margin,
                                    int32_t *__restrict__ d_bias, unsigned *d_status)
{
    const int lane = threadIdx.x;
    int cur = *d_cursor;
    cur = (cur < 0 || cur >= len) ? 0 : cur;
    const uint32_t fresh = __float_as_uint(*d_amax_new) & 0x7FFFFFFFu;
    uint32_t m = 0;
    for (int i = lane; i < len; i += 32) {
        uint32_t v = i == cur ? fresh : (__float_as_uint(d_history[i]) & 0x7FFFFFFFu);
        m = max(m, v);
    }
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    __syncwarp();
    if (lane == 0) {
        d_history[cur] = __uint_as_float(fresh);
        *d_cursor = cur + 1 == len ? 0 : cur + 1;
        unsigned flags = 0;
        *d_bias = bias_from_amax_bits(m, fmt, conv, margin, &flags);
        if (flags) atomicOr(d_status, flags);
    }
}

// Append `count` records {step, first_id + i, amax[i], bias[i]} to a ring of `capacity` records; *d_head counts
// every record ever appended (the slot of record n is n mod capacity).
__global__ void bias_log_kernel(fp8_bias_record_t *__restrict__ ring, int capacity, unsigned long long *d_head, int step,
                                int first_id, const float *__restrict__ d_amax, const int32_t *__restrict__ d_bias,
                                int count)
{
    const unsigned long long head = *d_head;
    for (int i = threadIdx.x; i < count; i += blockDim.x) {
        fp8_bias_record_t r;
        r.step = step;
        r.tensor_id = first_id + i;
        r.amax = d_amax[i];
        r.bias = d_bias[i];
        ring[(head + (unsigned long long)i) % (unsigned long long)capacity] = r;
    }
    __syncthreads();
    if (threadIdx.x == 0) *d_head = head + (unsigned long long)count;
}

// Mode of one tensor's bias over the records of the ring whose step lies in [step_lo, step_hi]: a histogram over
// every value Eq. 3 can produce for a 32-bit float amax (|bias| <= 165 with margins up to 16; others are counted
// but cannot win), the most frequent value wins, the smaller one on a tie.
constexpr int kModeLo = -192, kModeBins = 385;
__global__ void bias_mode_kernel(const fp8_bias_record_t *__restrict__ ring, int capacity,
                                 const unsigned long long *__restrict__ d_head, int tensor_id, int step_lo, int step_hi,
                                 int32_t *__restrict__ d_mode, int32_t *__restrict__ d_count, int32_t *__restrict__ d_samples)
{
    __shared__ unsigned hist[kModeBins];
    __shared__ unsigned samples;
    for (int i = threadIdx.x; i < kModeBins; i += blockDim.x) hist[i] = 0u;
    if (threadIdx.x == 0) samples = 0u;
    __syncthreads();
    const unsigned long long head = *d_head;
    const int valid = head < (unsigned long long)capacity ? (int)head : capacity;
    for (int i = threadIdx.x; i < valid; i += blockDim.x) {
        const fp8_bias_record_t r = ring[i];
        if (r.tensor_id == tensor_id && r.step >= step_lo && r.step <= step_hi) {
            atomicAdd(&samples, 1u);
            const int b = r.bias - kModeLo;
            if (b >= 0 && b < kModeBins) atomicAdd(&hist[b], 1u);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned best = 0u;
        int mode = 0;
        for (int i = 0; i < kModeBins; ++i)
            if (hist[i] > best) { best = hist[i]; mode = i + kModeLo; }
        *d_mode = mode;
        *d_count = (int32_t)best;
        if (d_samples) *d_samples = (int32_t)samples;
    }
}

template <int DT>
static cudaError_t launch_amax_rows(fp8_ctx *ctx, const void *x, int64_t rows, int64_t cols, int64_t ld, AmaxOut o,
                                    cudaStream_t stream)
{
    constexpr int kPerVec = DT == FP8_F32 ? 4 : 8;
    const bool aligned = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    const int max_blocks = ctx->sm_count * 6;
    int vec = (aligned && (ld % kPerVec) == 0) ? 1 : 0;
    int blocks = (int)(rows > max_blocks ? max_blocks : rows);
    count_launch();
    amax_rows_kernel<DT><<<blocks, kAmaxThreads, 0, stream>>>(x, rows, cols, ld, vec, o);
    return cudaGetLastError();
}

cudaError_t launch_amax_bias(fp8_ctx *ctx, const void *x, int dt, int64_t rows, int64_t cols, int64_t ld, float *d_amax,
                             int32_t *d_bias, int fmt, int conv, int margin, cudaStream_t stream)
{
    // contiguous and 16-byte aligned: the streaming kernel shared with fp8_cast_group, on one tensor
    if (ld == cols && (reinterpret_cast<uintptr_t>(x) & 15u) == 0 &&
        (rows * cols / 16) / 1024 < 0x7FFFFFFF)
        return launch_amax_flat(ctx, x, dt, rows * cols, d_amax, d_bias, fmt, conv, margin, stream);
    AmaxOut o{take_slot(ctx), d_amax, d_bias, ctx->d_status, fmt, conv, margin};
    if (dt == FP8_BF16) return launch_amax_rows<FP8_BF16>(ctx, x, rows, cols, ld, o, stream);
    if (dt == FP8_F16) return launch_amax_rows<FP8_F16>(ctx, x, rows, cols, ld, o, stream);
    return launch_amax_rows<FP8_F32>(ctx, x, rows, cols, ld, o, stream);
}

}  // namespace fp8lin

extern "C" {

fp8_status_t fp8_amax(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                      float *d_amax, void *stream)
{
    if (!ctx || !x || !d_amax) return FP8_ERR_NULL;
    if ((int)x_dt < 0 || (int)x_dt > 2) return FP8_ERR_DTYPE;
    if (rows <= 0 || cols <= 0 || ld < cols) return FP8_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(x) & (x_dt == FP8_F32 ? 3u : 1u)) return FP8_ERR_ALIGN;
    cudaError_t e = fp8lin::launch_amax_bias(ctx, x, (int)x_dt, rows, cols, ld, d_amax, nullptr, 0, 0, 0,
                                             (cudaStream_t)stream);
    return e == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_scaling_bias(fp8_ctx *ctx, const float *d_amax, fp8_format_t fmt, fp8_conv_t conv, int32_t margin,
                              int32_t *d_bias, void *stream)
{
    if (!ctx || !d_amax || !d_bias) return FP8_ERR_NULL;
    if ((int)fmt < 0 || (int)fmt > 1 || (int)conv < 0 || (int)conv > 1) return FP8_ERR_DTYPE;
    fp8lin::count_launch();
    fp8lin::scaling_bias_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(d_amax, (int)fmt, (int)conv, margin, d_bias,
                                                                  ctx->d_status);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_amax_history_bias(fp8_ctx *ctx, float *d_history, int32_t len, int32_t *d_cursor,
                                   const float *d_amax_new, fp8_format_t fmt, fp8_conv_t conv, int32_t margin,
                                   int32_t *d_bias, void *stream)
{
    if (!ctx || !d_history || !d_cursor || !d_amax_new || !d_bias) return FP8_ERR_NULL;
    if ((int)fmt < 0 || (int)fmt > 1 || (int)conv < 0 || (int)conv > 1) return FP8_ERR_DTYPE;
    if (len <= 0 || len > 65536) return FP8_ERR_SHAPE;
    fp8lin::count_launch();
    fp8lin::amax_history_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(d_history, len, d_cursor, d_amax_new, (int)fmt,
                                                                   (int)conv, margin, d_bias, ctx->d_status);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_bias_log_append(fp8_ctx *ctx, fp8_bias_record_t *d_ring, int32_t capacity, uint64_t *d_head, int32_t step,
                                 int32_t first_tensor_id, const float *d_amax, const int32_t *d_bias, int32_t count,
                                 void *stream)
{
    if (!ctx || !d_ring || !d_head || !d_amax || !d_bias) return FP8_ERR_NULL;
    if (capacity <= 0 || count <= 0 || count > capacity) return FP8_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_ring) & 3u) || (reinterpret_cast<uintptr_t>(d_head) & 7u)) return FP8_ERR_ALIGN;
    fp8lin::count_launch();
    fp8lin::bias_log_kernel<<<1, 128, 0, (cudaStream_t)stream>>>(d_ring, capacity,
                                                                reinterpret_cast<unsigned long long *>(d_head), step,
                                                                first_tensor_id, d_amax, d_bias, count);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_bias_mode(fp8_ctx *ctx, const fp8_bias_record_t *d_ring, int32_t capacity, const uint64_t *d_head,
                           int32_t tensor_id, int32_t step_lo, int32_t step_hi, int32_t *d_mode, int32_t *d_count,
                           int32_t *d_samples, void *stream)
{
    if (!ctx || !d_ring || !d_head || !d_mode || !d_count) return FP8_ERR_NULL;
    if (capacity <= 0 || step_lo > step_hi) return FP8_ERR_SHAPE;
    fp8lin::count_launch();
    fp8lin::bias_mode_kernel<<<1, 256, 0, (cudaStream_t)stream>>>(d_ring, capacity,
                                                                 reinterpret_cast<const unsigned long long *>(d_head),
                                                                 tensor_id, step_lo, step_hi, d_mode, d_count, d_samples);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

}  // extern "C"
