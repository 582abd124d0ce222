// fp8_amax_noalloc: the amax reduction for callers that cannot allocate.
//
// Some programs hand every byte of device memory to their own allocator at
// start-up, or run inside a host application that forbids cudaMalloc on its
// threads (it serialises against all streams of the device), or are plug-ins
// that are simply not given an allocator.  Such callers cannot create an
// fp8_ctx, because fp8_create allocates the reduction workspace.  This entry
// point needs no context and no allocation at all: its workspace is a
// fixed-size array that lives in the library's own device image.
//
// The price is a size limit and shared state:
//   - one partial maximum per 65 536-element chunk, kMaxChunks chunks, so at
//     most kMaxElements elements per call (larger tensors are rejected);
//   - every GPU that loads the library carries the 32 KiB array until exit;
//   - all calls on a device share it, so two calls whose kernels may overlap
//     on the GPU (different streams, no ordering between them) race.  Order
//     them on one stream or with events.
#include "fp8lin_internal.cuh"

namespace fp8lin {

constexpr int kNaThreads = 256;
constexpr int kNaUnroll = 4;
constexpr int64_t kChunkElems = 65536;             // 128 KiB of bf16 per partial
constexpr int kMaxChunks = 8192;
constexpr int64_t kMaxElements = kChunkElems * kMaxChunks;  // 2^29 elements = 1 GiB of bf16
constexpr int kMaxDevices = 64;

// [0, kMaxChunks): per-chunk partial maxima, rewritten by every call before
// they are read.  [kMaxChunks]: arrival counter, zero between calls (device
// images start zeroed; the last block of each call puts it back to zero).
static __device__ __align__(256) unsigned g_noalloc_scratch[kMaxChunks + 64];

__global__ void __launch_bounds__(kNaThreads)
amax_noalloc_kernel(const uint4 *__restrict__ x, int64_t nvec, int nchunks, const uint16_t *__restrict__ tail,
                    int ntail, unsigned *__restrict__ scratch, float *__restrict__ d_amax)
{
    __shared__ uint32_t warp_max[kNaThreads / 32];
    __shared__ bool is_last;
    const int64_t vec_per_chunk = kChunkElems / 8;
    for (int chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
        const int64_t v0 = (int64_t)chunk * vec_per_chunk;
        const int64_t v1 = min(nvec, v0 + vec_per_chunk);
        uint32_t acc = 0;
        for (int64_t base = v0; base < v1; base += (int64_t)kNaThreads * kNaUnroll) {
            uint4 v[kNaUnroll];
#pragma unroll
            for (int j = 0; j < kNaUnroll; ++j) {
                int64_t i = base + threadIdx.x + (int64_t)j * kNaThreads;
                v[j] = (i < v1) ? __ldg(x + i) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < kNaUnroll; ++j) {
                acc = __vmaxu2(acc, v[j].x & 0x7FFF7FFFu);
                acc = __vmaxu2(acc, v[j].y & 0x7FFF7FFFu);
                acc = __vmaxu2(acc, v[j].z & 0x7FFF7FFFu);
                acc = __vmaxu2(acc, v[j].w & 0x7FFF7FFFu);
            }
        }
        // the scalar tail (fewer than 8 elements) belongs to the last chunk
        if (chunk == nchunks - 1 && (int)threadIdx.x < ntail) acc = __vmaxu2(acc, (uint32_t)tail[threadIdx.x] & 0x7FFFu);
        uint32_t m = max(acc & 0xFFFFu, acc >> 16);
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int i = 1; i < kNaThreads / 32; ++i) m = max(m, warp_max[i]);
            scratch[chunk] = m;
        }
        __syncthreads();
    }
    // last block to finish folds the partials
    if (threadIdx.x == 0) {
        __threadfence();
        unsigned arrived = atomicAdd(&scratch[kMaxChunks], 1u) + 1u;
        is_last = (arrived == gridDim.x);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    uint32_t m = 0;
    for (int i = threadIdx.x; i < nchunks; i += kNaThreads) m = max(m, __ldcg(scratch + i));
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 1; i < kNaThreads / 32; ++i) m = max(m, warp_max[i]);
        *d_amax = __uint_as_float(m << 16);
        scratch[kMaxChunks] = 0u;  // ready for the next call
    }
}

// Device address of the scratch array, looked up once per device.  In host
// code the array's name is only a handle for the runtime, not an address a
// kernel could use, hence cudaGetSymbolAddress with that device current.
static unsigned *g_scratch_ptr[kMaxDevices];

static fp8_status_t scratch_for_current_device(unsigned **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FP8_ERR_CUDA;
    if (!g_scratch_ptr[dev]) {
        unsigned *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_noalloc_scratch) != cudaSuccess || !p) return FP8_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return FP8_OK;
}

}  // namespace fp8lin

extern "C" fp8_status_t fp8_amax_noalloc(const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                                         float *d_amax, void *stream)
{
    using namespace fp8lin;
    if (!x || !d_amax) return FP8_ERR_NULL;
    if ((int)x_dt < 0 || (int)x_dt > 2) return FP8_ERR_DTYPE;
    if (x_dt != FP8_BF16) return FP8_ERR_UNSUPPORTED;
    if (rows <= 0 || cols <= 0 || ld < cols) return FP8_ERR_SHAPE;
    if (ld != cols) return FP8_ERR_UNSUPPORTED;  // contiguous tensors only
    if (reinterpret_cast<uintptr_t>(x) & 15u) return FP8_ERR_ALIGN;
    if (rows > kMaxElements / cols || rows * cols > kMaxElements) return FP8_ERR_TOO_LARGE;
    unsigned *scratch = nullptr;
    fp8_status_t st = scratch_for_current_device(&scratch);
    if (st != FP8_OK) return st;
    const int64_t n = rows * cols;
    const int64_t nvec = n / 8;
    const int ntail = (int)(n - nvec * 8);
    int nchunks = (int)((n + kChunkElems - 1) / kChunkElems);
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return FP8_ERR_CUDA;
    int grid = nchunks < sms * 8 ? nchunks : sms * 8;
    amax_noalloc_kernel<<<grid, kNaThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const uint4 *>(x), nvec, nchunks, reinterpret_cast<const uint16_t *>(x) + nvec * 8, ntail,
        scratch, d_amax);
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}
