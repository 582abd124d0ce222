// Context, status reporting and the host-side scaling-bias helper.
#include <new>

#include "fp8lin_internal.cuh"

namespace fp8lin {
cudaError_t configure_gemm_kernels(int max_smem_optin);  // gemm.cu
std::atomic<unsigned long long> g_kernel_launches{0};
}

extern "C" {

fp8_status_t fp8_launch_count(uint64_t *count)
{
    if (!count) return FP8_ERR_NULL;
    *count = (uint64_t)fp8lin::g_kernel_launches.load(std::memory_order_relaxed);
    return FP8_OK;
}

const char *fp8_status_string(fp8_status_t s)
{
    switch (s) {
    case FP8_OK: return "ok";
    case FP8_ERR_NULL: return "required pointer is NULL";
    case FP8_ERR_SHAPE: return "bad shape";
    case FP8_ERR_ALIGN: return "pointer or leading dimension not aligned as required";
    case FP8_ERR_DTYPE: return "bad enum value";
    case FP8_ERR_UNSUPPORTED: return "no kernel for this request";
    case FP8_ERR_CUDA: return "CUDA call failed";
    case FP8_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case FP8_ERR_TOO_LARGE: return "tensor exceeds the fixed workspace of the no-allocation entry point";
    }
    return "unknown status";
}

fp8_status_t fp8_create(fp8_ctx **out, int device)
{
    if (!out) return FP8_ERR_NULL;
    *out = nullptr;
    if (cudaSetDevice(device) != cudaSuccess) return FP8_ERR_CUDA;
    fp8_ctx *ctx = new (std::nothrow) fp8_ctx();
    if (!ctx) return FP8_ERR_CUDA;
    ctx->device = device;
    ctx->next_slot = 0;
    bool ok = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) == cudaSuccess &&
              cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) ==
                  cudaSuccess;
    int major = 0;
    ok = ok && cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) == cudaSuccess;
    if (!ok) { delete ctx; return FP8_ERR_CUDA; }
    if (major != 10) { delete ctx; return FP8_ERR_UNSUPPORTED; }  // sm_100a code only

    size_t words = 1 + (size_t)fp8lin::kReduceSlots * fp8lin::kSlotWords + 2;
    unsigned *buf = nullptr;
    if (cudaMalloc(&buf, words * sizeof(unsigned)) != cudaSuccess) { delete ctx; return FP8_ERR_CUDA; }
    if (cudaMemset(buf, 0, words * sizeof(unsigned)) != cudaSuccess) { cudaFree(buf); delete ctx; return FP8_ERR_CUDA; }
    ctx->d_status = buf;
    ctx->d_slots = buf + 1;
    ctx->d_predict_stats = buf + 1 + fp8lin::kReduceSlots * fp8lin::kSlotWords;
    ctx->partial_bytes = (size_t)64 << 20;
    ctx->d_partial = nullptr;
    if (cudaMalloc(&ctx->d_partial, ctx->partial_bytes) != cudaSuccess) { cudaFree(buf); delete ctx; return FP8_ERR_CUDA; }

    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaFree(ctx->d_partial);
        cudaFree(buf);
        delete ctx;
        return FP8_ERR_CUDA;
    }
    ctx->encode_tiled = (fp8lin::EncodeTiledFn)fn;
    if (fp8lin::configure_gemm_kernels(ctx->max_smem_optin) != cudaSuccess) {
        cudaFree(ctx->d_partial);
        cudaFree(buf);
        delete ctx;
        return FP8_ERR_CUDA;
    }
    *out = ctx;
    return FP8_OK;
}

fp8_status_t fp8_destroy(fp8_ctx *ctx)
{
    if (!ctx) return FP8_ERR_NULL;
    cudaSetDevice(ctx->device);
    cudaError_t e = cudaFree(ctx->d_status);
    cudaError_t e2 = cudaFree(ctx->d_partial);
    if (e == cudaSuccess) e = e2;
    delete ctx;
    return e == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_device_flags(fp8_ctx *ctx, void *stream, unsigned *flags, int clear)
{
    if (!ctx || !flags) return FP8_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(flags, ctx->d_status, sizeof(unsigned), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return FP8_ERR_CUDA;
    if (clear && cudaMemsetAsync(ctx->d_status, 0, sizeof(unsigned), st) != cudaSuccess) return FP8_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FP8_ERR_CUDA;
    return (*flags & FP8_FLAG_TIMEOUT) ? FP8_ERR_DEVICE_TIMEOUT : FP8_OK;
}

fp8_status_t fp8_scaling_bias_host(float amax, fp8_format_t fmt, fp8_conv_t conv, int32_t margin, int32_t *bias)
{
    if (!bias) return FP8_ERR_NULL;
    if ((int)fmt < 0 || (int)fmt > 1 || (int)conv < 0 || (int)conv > 1) return FP8_ERR_DTYPE;
    uint32_t bits;
    __builtin_memcpy(&bits, &amax, 4);
    unsigned flags = 0;
    *bias = fp8lin::bias_from_amax_bits(bits, (int)fmt, (int)conv, margin, &flags);
    return FP8_OK;
}

}  // extern "C"
