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

// Input element types: bytes per element and words per group of four elements.
template <int DT>
struct InType {
    static constexpr int kBytes = (DT == FP8_F32) ? 4 : 2;
    static constexpr int kWords4 = (DT == FP8_F32) ? 4 : 2;
};

// Four consecutive input elements (kWords4 words, memory order) as floats; every conversion is exact.
template <int DT>
__device__ __forceinline__ void unpack4(const uint32_t *w, float (&f)[4])
{
    if (DT == FP8_BF16) {
        f[0] = __uint_as_float(w[0] << 16);
        f[1] = __uint_as_float(w[0] & 0xFFFF0000u);
        f[2] = __uint_as_float(w[1] << 16);
        f[3] = __uint_as_float(w[1] & 0xFFFF0000u);
    } else if (DT == FP8_F16) {
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; cvt.f32.f16 %0, lo; cvt.f32.f16 %1, hi; }"
            : "=f"(f[0]), "=f"(f[1]) : "r"(w[0]));
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; cvt.f32.f16 %0, lo; cvt.f32.f16 %1, hi; }"
            : "=f"(f[2]), "=f"(f[3]) : "r"(w[1]));
    } else {
        f[0] = __uint_as_float(w[0]);
        f[1] = __uint_as_float(w[1]);
        f[2] = __uint_as_float(w[2]);
        f[3] = __uint_as_float(w[3]);
    }
}

// Scale four values by the exact power of two and round them to four FP8 bytes (memory order).
template <int FMT, bool TWO_STEP>
__device__ __forceinline__ uint32_t pack4(float (&f)[4], Pow2Pair p, bool &sat)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[i] *= p.first;
        if (TWO_STEP) f[i] *= p.second;
    }
    sat = sat || clips<FMT>(f[0]) || clips<FMT>(f[1]) || clips<FMT>(f[2]) || clips<FMT>(f[3]);
    return cvt_pair<FMT>(f[1], f[0]) | (cvt_pair<FMT>(f[3], f[2]) << 16);
}

template <int FMT, int DT, bool TWO_STEP>
__device__ __forceinline__ uint32_t cast4w(const uint32_t *w, Pow2Pair p, bool &sat)
{
    float f[4];
    unpack4<DT>(w, f);
    return pack4<FMT, TWO_STEP>(f, p, sat);
}

// Four bf16 values (two packed words, memory order) -> four FP8 bytes (memory order).
template <int FMT, bool TWO_STEP>
__device__ __forceinline__ uint32_t cast4(uint32_t w0, uint32_t w1, Pow2Pair p, bool &sat)
{
    const uint32_t w[2] = {w0, w1};
    return cast4w<FMT, FP8_BF16, TWO_STEP>(w, p, sat);
}

// Element i of a tensor of type DT as a float (exact).
template <int DT>
__device__ __forceinline__ float load1(const void *x, int64_t i)
{
    if (DT == FP8_F32) return reinterpret_cast<const float *>(x)[i];
    const uint16_t h = reinterpret_cast<const uint16_t *>(x)[i];
    if (DT == FP8_BF16) return __uint_as_float((uint32_t)h << 16);
    float f;
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"(h));
    return f;
}

template <int FMT, int DT, bool TWO_STEP>
__device__ __forceinline__ uint8_t cast1(const void *x, int64_t i, Pow2Pair p, bool &sat)
{
    float f = load1<DT>(x, i) * p.first;
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


}  // namespace fp8lin
