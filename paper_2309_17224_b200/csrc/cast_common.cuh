// Conversion helpers shared by the cast kernels.
#pragma once

#include "fp8lin_internal.cuh"

namespace fp8lin {

constexpr int kCastThreads = 256;

template <int FMT>
__device__ __forceinline__ uint32_t cvt_pair(float hi, float lo)
{
    uint16_t r;
    if (FMT == FP8_E4)
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else
        asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return (uint32_t)r;
}

// True when RNE to the format would land beyond its largest finite value.
template <int FMT>
__device__ __forceinline__ bool clips(float v)
{
    return FMT == FP8_E4 ? (fabsf(v) > 464.0f) : (fabsf(v) >= 61440.0f);
}

// Four bf16 values (two packed words, memory order) -> four FP8 bytes (memory order).
template <int FMT, bool TWO_STEP>
__device__ __forceinline__ uint32_t cast4(uint32_t w0, uint32_t w1, Pow2Pair p, bool &sat)
{
    float f0 = __uint_as_float(w0 << 16) * p.first;
    float f1 = __uint_as_float(w0 & 0xFFFF0000u) * p.first;
    float f2 = __uint_as_float(w1 << 16) * p.first;
    float f3 = __uint_as_float(w1 & 0xFFFF0000u) * p.first;
    if (TWO_STEP) { f0 *= p.second; f1 *= p.second; f2 *= p.second; f3 *= p.second; }
    sat = sat || clips<FMT>(f0) || clips<FMT>(f1) || clips<FMT>(f2) || clips<FMT>(f3);
    return cvt_pair<FMT>(f1, f0) | (cvt_pair<FMT>(f3, f2) << 16);
}

template <int FMT, bool TWO_STEP>
__device__ __forceinline__ uint8_t cast1(uint16_t h, Pow2Pair p, bool &sat)
{
    float f = __uint_as_float((uint32_t)h << 16) * p.first;
    if (TWO_STEP) f *= p.second;
    sat = sat || clips<FMT>(f);
    return (uint8_t)(cvt_pair<FMT>(0.0f, f) & 0xFFu);
}

// Transpose a 4x4 byte block held as four row words into four column words.
__device__ __forceinline__ void transpose4x4(const uint32_t r[4], uint32_t c[4])
{
    uint32_t t0 = __byte_perm(r[0], r[1], 0x5140);
    uint32_t t1 = __byte_perm(r[2], r[3], 0x5140);
    uint32_t t2 = __byte_perm(r[0], r[1], 0x7362);
    uint32_t t3 = __byte_perm(r[2], r[3], 0x7362);
    c[0] = __byte_perm(t0, t1, 0x5410);
    c[1] = __byte_perm(t0, t1, 0x7632);
    c[2] = __byte_perm(t2, t3, 0x5410);
    c[3] = __byte_perm(t2, t3, 0x7632);
}


// Launches the fused single-launch amax + bias + cast (cast_fused.cu).  Returns cudaErrorNotSupported when the
// tensor does not meet its shape rules, in which case the caller uses the two-launch path.
cudaError_t launch_cast_fused(fp8_ctx *ctx, int fmt, const void *x, int64_t rows, int64_t cols, int64_t ld, int conv,
                              int margin, float *d_amax_out, int32_t *d_bias_out, uint8_t *y, uint8_t *y_t,
                              cudaStream_t stream);

}  // namespace fp8lin
