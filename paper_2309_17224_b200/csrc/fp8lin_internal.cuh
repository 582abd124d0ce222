// Internal declarations shared by the translation units of libfp8lin.so.
#pragma once

#include <atomic>

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fp8lin.h"

namespace fp8lin {

// ---------------------------------------------------------------------------
// context
// ---------------------------------------------------------------------------

constexpr int kReduceSlots = 64;   // independent grid-reduction slots, used round-robin
constexpr int kSlotWords = 4;      // {running max, arrival counter, scratch flag, redo flag of a predicted cast}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace fp8lin

struct fp8_ctx {
    int device;
    int sm_count;
    int max_smem_optin;
    unsigned *d_status;   // one sticky word of FP8_FLAG_* bits
    unsigned *d_slots;    // kReduceSlots * kSlotWords words, all zero between calls
    unsigned next_slot;
    unsigned *d_predict_stats;   // {guesses that held, guesses that did not} of fp8_cast_predicted
    float *d_partial;     // FP32 workspace for split-K partial sums
    size_t partial_bytes;
    fp8lin::EncodeTiledFn encode_tiled;
};

namespace fp8lin {

inline unsigned *take_slot(fp8_ctx *ctx)
{
    unsigned s = ctx->next_slot++ % kReduceSlots;
    return ctx->d_slots + s * kSlotWords;
}

// Format shift between the paper-convention bias and the shift that yields
// native bytes (+1 for E4 under the paper convention, else 0).
__host__ __device__ inline int format_delta(int fmt, int conv)
{
    return (fmt == FP8_E4 && conv == FP8_CONV_PAPER) ? 1 : 0;
}

// Eq. 3 on the bits of a non-negative float: the largest b with
// amax * 2^b <= max_num, minus margin.  max_num = m_max * 2^e_max with
// (1.875, 7) for 240, (1.75, 8) for 448, (1.75, 15) for 57344.
__host__ __device__ inline int bias_from_amax_bits(uint32_t bits, int fmt, int conv, int margin, unsigned *flags)
{
    bits &= 0x7FFFFFFFu;
    if (bits == 0u) { *flags |= FP8_FLAG_ZERO_AMAX; return 0; }
    if (bits >= 0x7F800000u) { *flags |= FP8_FLAG_NONFINITE_AMAX; return 0; }
    int e;
    uint32_t frac;  // 23 fraction bits of the normalised significand
    uint32_t ef = bits >> 23;
    uint32_t mant = bits & 0x7FFFFFu;
    if (ef != 0u) {
        e = (int)ef - 127;
        frac = mant;
    } else {  // subnormal: normalise
        int hb = 22;
        while (((mant >> hb) & 1u) == 0u) --hb;
        e = -149 + hb;
        frac = (mant << (23 - hb)) & 0x7FFFFFu;
    }
    int e_max;
    uint32_t frac_max;
    if (fmt == FP8_E5) { e_max = 15; frac_max = 0x600000u; }
    else if (conv == FP8_CONV_PAPER) { e_max = 7; frac_max = 0x700000u; }
    else { e_max = 8; frac_max = 0x600000u; }
    return e_max - e - (frac > frac_max ? 1 : 0) - margin;
}

// Kernels this library has launched in this process (fp8_launch_count); bumped beside every launch.
extern std::atomic<unsigned long long> g_kernel_launches;
inline void count_launch(int n = 1) { g_kernel_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// Launch allowed to start while the launch before it on the stream drains (programmatic dependent launch); the
// kernel itself waits (griddepcontrol.wait) before it touches anything an earlier launch may have written.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t stream,
                                    Args... args)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

cudaError_t launch_amax_bias(fp8_ctx *ctx, const void *x, int dt, int64_t rows, int64_t cols, int64_t ld, float *d_amax,
                             int32_t *d_bias, int fmt, int conv, int margin, cudaStream_t stream);

// group.cu: the streaming kernels of fp8_cast_group applied to one contiguous, 16-byte aligned tensor of n elements
cudaError_t launch_amax_flat(fp8_ctx *ctx, const void *x, int dt, int64_t n, float *d_amax, int32_t *d_bias, int fmt,
                             int conv, int margin, cudaStream_t st);
cudaError_t launch_cast_flat(fp8_ctx *ctx, const void *x, int dt, int64_t n, const int32_t *d_bias, int fmt, int delta,
                             uint8_t *y, cudaStream_t st);
cudaError_t launch_one_pass_flat(fp8_ctx *ctx, const void *x, int dt, int64_t n, int fmt, int conv, int margin,
                                 float *d_amax, const int32_t *d_bias_in, int32_t *d_bias_out, int verify, uint8_t *y,
                                 cudaStream_t st);

}  // namespace fp8lin

// ---------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------
#ifdef __CUDACC__
namespace fp8lin {

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// 2^e as a float for e in [-126, 127].
__device__ __forceinline__ float pow2_normal(int e)
{
    return __uint_as_float((uint32_t)(e + 127) << 23);
}

// x * 2^s split into two exact power-of-two factors so that any s in
// [-300, 300] works: the first factor carries as much of s as one normal
// float can, the second the rest.
struct Pow2Pair {
    float first, second;
};
__device__ __forceinline__ Pow2Pair make_pow2_pair(int s)
{
    int s1 = max(-126, min(127, s));
    int s2 = max(-126, min(127, s - s1));
    Pow2Pair p;
    p.first = pow2_normal(s1);
    p.second = pow2_normal(s2);
    return p;
}

}  // namespace fp8lin
#endif
