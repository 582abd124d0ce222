// Scale-and-cast (Eq. 1 followed by the cast of Section 2.1; E5 per Section
// 2.2) and post-training quantisation of a weight tensor (Section 3.1).
//
// code = RNE_fp8(x * 2^(bias + delta)), saturating.  The input (bf16, fp16 or
// fp32) converts to FP32 exactly, the scaling is an exact power-of-two multiply
// (the product is exact unless it underflows FP32, where the FP8 result is zero
// either way) and the rounding is one hardware cvt.rn.satfinite per pair.
//
// Kernels, all HBM-bound (2 B read per 16-bit element + 1 B written per element and layout):
//   (group.cu)             contiguous tensor, row-major output: the streaming kernels shared with
//                          fp8_cast_group -- cast, amax + cast in one pass (fp8_cast_predicted, delayed scaling).
//   cast_tile_kernel       128x128 tiles, optional row-major output and optional transposed output
//                          staged through shared memory so that both are written in 128-byte rows;
//                          also the guarded path for ragged or strided tensors.
//   cast_small_kernel      decode-size tensors: one cluster keeps the tensor in registers between
//                          its amax and its cast, one launch.
// The cast kernels walk the tensor from its end to its start: when the amax pass has just streamed
// it front to back, the part most recently read is the part most likely still in L2.
#include <cstdlib>

#include "cast_common.cuh"

namespace fp8lin {

// ---------------------------------------------------------------------------
// tiled, with optional transposed output
// ---------------------------------------------------------------------------

constexpr int kTile = 128;

template <int FMT, int DT>
__global__ void __launch_bounds__(kCastThreads) cast_tile_kernel(const void *__restrict__ x, int64_t rows,
                                                                 int64_t cols, int64_t ld,
                                                                 const int32_t *__restrict__ d_bias, int delta,
                                                                 uint8_t *__restrict__ y, uint8_t *__restrict__ y_t,
                                                                 int fast_ok, unsigned *d_status)
{
    // Transposed staging: word (c, w) holds rows 4w..4w+3 of tile column c; the
    // word position is rotated by c/4 so that both the column-wise writes and
    // the row-wise reads touch 32 distinct banks.
    __shared__ uint32_t stage[kTile][kTile / 4];
    constexpr int kW = InType<DT>::kWords4;  // words per four input elements
    constexpr int kB = InType<DT>::kBytes;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // see cast_flat_kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int s = __ldcg(d_bias) + delta;   // at L2: the word may come from the launch before this one (see ptx.cuh)
    const Pow2Pair p = make_pow2_pair(s);
    bool sat = false;

    const int64_t tiles_c = (cols + kTile - 1) / kTile;
    const int64_t tile = (int64_t)gridDim.x - 1 - blockIdx.x;
    const int64_t r0 = (tile / tiles_c) * kTile;
    const int64_t c0 = (tile % tiles_c) * kTile;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (fast_ok && r0 + kTile <= rows && c0 + kTile <= cols) {
        uint32_t v[4][4][kW];
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int rg = warp + 8 * it;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint8_t *src = reinterpret_cast<const uint8_t *>(x) + ((r0 + 4 * rg + i) * ld + c0 + 4 * lane) * kB;
                if (kW == 2) {
                    const uint2 q = __ldcs(reinterpret_cast<const uint2 *>(src));
                    v[it][i][0] = q.x; v[it][i][1] = q.y;
                } else {
                    const uint4 q = __ldcs(reinterpret_cast<const uint4 *>(src));
                    v[it][i][0] = q.x; v[it][i][1] = q.y; v[it][i][kW - 2] = q.z; v[it][i][kW - 1] = q.w;
                }
            }
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int rg = warp + 8 * it;
            uint32_t rw[4], cw[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) rw[i] = cast4w<FMT, DT, true>(v[it][i], p, sat);
            if (y) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    *reinterpret_cast<uint32_t *>(y + (r0 + 4 * rg + i) * cols + c0 + 4 * lane) = rw[i];
            }
            if (y_t) {
                transpose4x4(rw, cw);
#pragma unroll
                for (int j = 0; j < 4; ++j) stage[4 * lane + j][(rg + lane) & 31] = cw[j];
            }
        }
        if (y_t) {
            __syncthreads();
#pragma unroll 4
            for (int cc = warp; cc < kTile; cc += 8) {
                uint32_t w = stage[cc][(lane + (cc >> 2)) & 31];
                *reinterpret_cast<uint32_t *>(y_t + (c0 + cc) * rows + r0 + 4 * lane) = w;
            }
        }
    } else {
        // Guarded path for ragged tiles and unaligned tensors: one element at a time.
        uint8_t *stage_b = reinterpret_cast<uint8_t *>(&stage[0][0]);  // [c][r] bytes
        for (int idx = threadIdx.x; idx < kTile * kTile; idx += kCastThreads) {
            int r = idx / kTile, c = idx % kTile;
            if (r0 + r < rows && c0 + c < cols) {
                uint8_t code = cast1<FMT, DT, true>(x, (r0 + r) * ld + c0 + c, p, sat);
                if (y) y[(r0 + r) * cols + c0 + c] = code;
                if (y_t) stage_b[c * kTile + r] = code;
            }
        }
        if (y_t) {
            __syncthreads();
            for (int idx = threadIdx.x; idx < kTile * kTile; idx += kCastThreads) {
                int c = idx / kTile, r = idx % kTile;
                if (r0 + r < rows && c0 + c < cols) y_t[(c0 + c) * rows + r0 + r] = stage_b[c * kTile + r];
            }
        }
    }
    if (__syncthreads_or(sat) && threadIdx.x == 0) atomicOr(d_status, FP8_FLAG_SATURATED);
}

template <int FMT, int DT>
static cudaError_t launch_cast(fp8_ctx *ctx, const void *x, int64_t rows, int64_t cols, int64_t ld,
                               const int32_t *d_bias, int delta, uint8_t *y, uint8_t *y_t, cudaStream_t stream)
{
    auto al = [](const void *p, unsigned a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
    constexpr int kB = InType<DT>::kBytes;
    if (!y_t && ld == cols && al(x, 16) && al(y, 16))   // the streaming kernel shared with fp8_cast_group, on one tensor
        return launch_cast_flat(ctx, x, DT, rows * cols, d_bias, FMT, delta, y, stream);
    int fast_ok = al(x, 4 * kB) && (ld % 4) == 0 && (!y || (al(y, 4) && (cols % 4) == 0)) &&
                  (!y_t || (al(y_t, 4) && (rows % 4) == 0));
    int64_t tiles = ((rows + kTile - 1) / kTile) * ((cols + kTile - 1) / kTile);
    if (tiles > 0x7FFFFFFF) return cudaErrorInvalidValue;
    return launch_dependent(cast_tile_kernel<FMT, DT>, (unsigned)tiles, kCastThreads, stream, x, rows, cols, ld, d_bias, delta,
                            y, y_t, fast_ok, ctx->d_status);
}

template <int FMT>
static cudaError_t launch_cast_dt(int dt, fp8_ctx *ctx, const void *x, int64_t rows, int64_t cols, int64_t ld,
                                  const int32_t *d_bias, int delta, uint8_t *y, uint8_t *y_t, cudaStream_t stream)
{
    if (dt == FP8_BF16) return launch_cast<FMT, FP8_BF16>(ctx, x, rows, cols, ld, d_bias, delta, y, y_t, stream);
    if (dt == FP8_F16) return launch_cast<FMT, FP8_F16>(ctx, x, rows, cols, ld, d_bias, delta, y, y_t, stream);
    return launch_cast<FMT, FP8_F32>(ctx, x, rows, cols, ld, d_bias, delta, y, y_t, stream);
}

// ---------------------------------------------------------------------------
// FP8-AMAX in one pass when the bias can be guessed
// ---------------------------------------------------------------------------
//
// Section 3 names the cost of just-in-time scaling (a second pass over memory) and the usual remedy (reuse the
// amax history).  Scaling biases change rarely between training steps (Appendix I: weights and activations
// almost never, gradients early on), so this kernel casts with a GUESS of the bias -- whatever the caller left in
// the bias word, typically the previous step's value -- while it takes the amax of the same pass.  The last block
// derives the true bias; if the guess was right the bytes already written are the exact FP8-AMAX result and the
// second launch (the ordinary cast, gated on a flag) returns at once.  If it was wrong the second launch redoes
// the cast with the true bias.  Either way the outputs equal fp8_cast_* with d_bias = NULL, bit for bit.
// Traffic: 2 B read + 1 B written per element when the guess holds, twice that when it does not.

template <int FMT, int DT>
static cudaError_t launch_predicted(fp8_ctx *ctx, const void *x, int64_t n, int conv, int margin, float *d_amax,
                                    const int32_t *d_bias_in, int32_t *d_bias_inout, int verify, uint8_t *y,
                                    cudaStream_t stream)
{
    // the one-pass kernel of group.cu on one tensor, followed (when the guess is verified) by the gated cast pass
    return launch_one_pass_flat(ctx, x, DT, n, FMT, conv, margin, d_amax, d_bias_in, d_bias_inout, verify, y, stream);
}

// ---------------------------------------------------------------------------
// small tensors: FP8-AMAX in one launch, the tensor held in registers
// ---------------------------------------------------------------------------
//
// Decode-size activations (a few tokens x hidden size) are far too small to fill the GPU, and two launches
// plus a grid-level reduction cost more than the work.  Here one thread-block cluster of one or two CTAs loads
// the whole tensor into registers (at most eight 16-byte vectors per thread), reduces the amax through shared
// memory and across the cluster through distributed shared memory, and casts from the registers: one launch,
// 2 B read + 1 B written per element, no global scratch.

constexpr int kSmallThreads = 1024;
constexpr int kSmallVecs = 8;          // 16-byte vectors per thread
#ifndef FP8LIN_SMALL_MAX_CTAS
#define FP8LIN_SMALL_MAX_CTAS 2
#endif
constexpr int kSmallMaxCtas = FP8LIN_SMALL_MAX_CTAS;   // beyond ~128K elements the two-launch path (whole GPU) is faster

template <int FMT, int DT>
__global__ void __launch_bounds__(kSmallThreads)
cast_small_kernel(const uint4 *__restrict__ x, uint4 *__restrict__ y, int64_t nvec, int ntail, int fmt, int conv,
                  int margin, int delta, float *d_amax, int32_t *d_bias, unsigned *d_status)
{
    constexpr int kPerVec = 16 / InType<DT>::kBytes;     // input elements per 16-byte vector
    constexpr int kW = InType<DT>::kWords4;
    __shared__ uint32_t warp_max[kSmallThreads / 32];
    __shared__ uint32_t cta_max;
    uint32_t rank, nctas;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(nctas));
    const int64_t stride = (int64_t)nctas * kSmallThreads;
    const int64_t t0 = (int64_t)rank * kSmallThreads + threadIdx.x;
    // A matmul launched behind this kernel as a programmatic dependent may take its places now and start
    // streaming its weights; it waits for this grid to complete before it touches anything written here.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the tensor may come from the launch before this one

    uint4 v[kSmallVecs];
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < kSmallVecs; ++j) {
        const int64_t i = t0 + j * stride;
        v[j] = i < nvec ? __ldcs(x + i) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int j = 0; j < kSmallVecs; ++j) {
        const uint32_t *w = reinterpret_cast<const uint32_t *>(&v[j]);
#pragma unroll
        for (int k = 0; k < 4; ++k) acc = DT == FP8_F32 ? max(acc, w[k] & 0x7FFFFFFFu) : __vmaxu2(acc, w[k] & 0x7FFF7FFFu);
    }
    if (rank == 0 && (int)threadIdx.x < ntail) {
        const int64_t i = nvec * kPerVec + threadIdx.x;
        if (DT == FP8_F32) acc = max(acc, reinterpret_cast<const uint32_t *>(x)[i] & 0x7FFFFFFFu);
        else acc = __vmaxu2(acc, (uint32_t)reinterpret_cast<const uint16_t *>(x)[i] & 0x7FFFu);
    }
    uint32_t m = DT == FP8_F32 ? acc : max(acc & 0xFFFFu, acc >> 16);
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = warp_max[threadIdx.x];
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        if (threadIdx.x == 0) cta_max = m;
    }
    // every CTA's maximum becomes visible to the whole cluster, then each CTA folds all of them
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    uint32_t total = 0;
    for (uint32_t r = 0; r < nctas; ++r) {
        uint32_t remote, val;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(&cta_max)), "r"(r));
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(val) : "r"(remote) : "memory");
        total = max(total, val);
    }
    uint32_t fbits;
    if (DT == FP8_F32) fbits = total;
    else if (DT == FP8_BF16) fbits = total << 16;
    else { float f; asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"((uint16_t)total)); fbits = __float_as_uint(f); }
    unsigned flags = 0;
    const int bias = bias_from_amax_bits(fbits, fmt, conv, margin, &flags);
    if (rank == 0 && threadIdx.x == 0) {
        *d_amax = __uint_as_float(fbits);
        *d_bias = bias;
        if (flags) atomicOr(d_status, flags);
    }
    const Pow2Pair p = make_pow2_pair(bias + delta);
    bool sat = false;
    // two input vectors (16-bit types) or four (fp32) make one 16-byte output vector
    constexpr int kIn = InType<DT>::kBytes;
#pragma unroll
    for (int j = 0; j < kSmallVecs; ++j) {
        const int64_t i = t0 + j * stride;
        if (i >= nvec) continue;
        const uint32_t *w = reinterpret_cast<const uint32_t *>(&v[j]);
        uint8_t *dst = reinterpret_cast<uint8_t *>(y) + i * kPerVec;
        if (kIn == 2) {
            uint2 o;
            o.x = cast4w<FMT, DT, true>(w, p, sat);
            o.y = cast4w<FMT, DT, true>(w + kW, p, sat);
            *reinterpret_cast<uint2 *>(dst) = o;
        } else {
            *reinterpret_cast<uint32_t *>(dst) = cast4w<FMT, DT, true>(w, p, sat);
        }
    }
    if (rank == 0 && (int)threadIdx.x < ntail) {
        const int64_t i = nvec * kPerVec + threadIdx.x;
        reinterpret_cast<uint8_t *>(y)[i] = cast1<FMT, DT, true>(x, i, p, sat);
    }
    if (__syncthreads_or(sat) && threadIdx.x == 0) atomicOr(d_status, FP8_FLAG_SATURATED);
    // no CTA may exit while a peer can still read its cta_max
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int FMT, int DT>
static cudaError_t launch_small(fp8_ctx *ctx, const void *x, int64_t n, int conv, int margin, float *d_amax,
                                int32_t *d_bias, uint8_t *y, cudaStream_t stream)
{
    constexpr int kPerVec = 16 / InType<DT>::kBytes;
    const int64_t nvec = n / kPerVec;
    const int ntail = (int)(n - nvec * kPerVec);
    const int64_t per_cta = (int64_t)kSmallThreads * kSmallVecs;
    int64_t want = (nvec + per_cta - 1) / per_cta;
    if (want > kSmallMaxCtas) return cudaErrorNotSupported;
    int ctas = 1;
    while (ctas < want) ctas *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    cfg.blockDim = dim3(kSmallThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)ctas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // may be set up while the launch before it drains; it reads nothing before that launch has completed
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    count_launch();
    return cudaLaunchKernelEx(&cfg, cast_small_kernel<FMT, DT>, reinterpret_cast<const uint4 *>(x),
                              reinterpret_cast<uint4 *>(y), nvec, ntail, (int)FMT, conv, margin, format_delta(FMT, conv),
                              d_amax, d_bias, ctx->d_status);
}

static cudaError_t launch_small_any(int fmt, int dt, fp8_ctx *ctx, const void *x, int64_t n, int conv, int margin,
                                    float *d_amax, int32_t *d_bias, uint8_t *y, cudaStream_t st)
{
#define FP8LIN_SMALL(F, D) return launch_small<F, D>(ctx, x, n, conv, margin, d_amax, d_bias, y, st)
    if (fmt == FP8_E4) {
        if (dt == FP8_BF16) FP8LIN_SMALL(FP8_E4, FP8_BF16);
        if (dt == FP8_F16) FP8LIN_SMALL(FP8_E4, FP8_F16);
        FP8LIN_SMALL(FP8_E4, FP8_F32);
    }
    if (dt == FP8_BF16) FP8LIN_SMALL(FP8_E5, FP8_BF16);
    if (dt == FP8_F16) FP8LIN_SMALL(FP8_E5, FP8_F16);
    FP8LIN_SMALL(FP8_E5, FP8_F32);
#undef FP8LIN_SMALL
}

// ---------------------------------------------------------------------------
// range statistics under a given bias
// ---------------------------------------------------------------------------
//
// The constant-bias experiments (FP8-CSCALE, Section 4 and Appendix F) ask which biases keep a tensor inside
// the FP8 range.  This kernel answers for one tensor and one bias without writing any bytes: how many elements
// would be clipped to the maximum, how many non-zero elements would be flushed to zero, how many would land in
// the subnormal range, out of how many non-zero finite elements.

template <int FMT, int DT>
__global__ void __launch_bounds__(256) range_stats_kernel(const void *__restrict__ x, int64_t rows, int64_t cols,
                                                          int64_t ld, const int32_t *__restrict__ d_bias, int delta,
                                                          unsigned long long *__restrict__ d_counts)
{
    const Pow2Pair p = make_pow2_pair(__ldg(d_bias) + delta);
    constexpr uint32_t kMantMask = FMT == FP8_E4 ? 0x07u : 0x03u;
    unsigned clipped = 0, flushed = 0, subnormal = 0, nonzero = 0;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        for (int64_t c = threadIdx.x; c < cols; c += blockDim.x) {
            const float xv = load1<DT>(x, r * ld + c);
            if (xv != xv) continue;                       // NaN: neither in nor out of range
            const bool finite_nz = xv != 0.0f && fabsf(xv) <= 3.402823466e38f;
            nonzero += finite_nz;
            const float v = xv * p.first * p.second;
            const uint32_t code = cvt_pair<FMT>(0.0f, v) & 0x7Fu;
            clipped += clips<FMT>(v);
            flushed += finite_nz && code == 0u;
            subnormal += code != 0u && (code & ~kMantMask) == 0u;
        }
    }
    unsigned vals[4] = {clipped, flushed, subnormal, nonzero};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        unsigned v = __reduce_add_sync(0xFFFFFFFFu, vals[i]);
        if ((threadIdx.x & 31) == 0 && v) atomicAdd(&d_counts[i], (unsigned long long)v);
    }
}

#ifdef FP8LIN_EXPERIMENTS
static const bool g_no_small_cast = [] { const char *e = getenv("FP8LIN_NO_SMALL_CAST"); return e && e[0] == '1'; }();
#else
constexpr bool g_no_small_cast = false;
#endif

static fp8_status_t cast_entry(int fmt, fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols,
                               int64_t ld, const int32_t *d_bias, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                               int32_t *d_bias_out, uint8_t *y, uint8_t *y_t, void *stream)
{
    if (!ctx || !x || (!y && !y_t)) return FP8_ERR_NULL;
    if (!d_bias && (!d_amax_out || !d_bias_out)) return FP8_ERR_NULL;
    if ((int)x_dt < 0 || (int)x_dt > 2 || (int)conv < 0 || (int)conv > 1) return FP8_ERR_DTYPE;
    if (rows <= 0 || cols <= 0 || ld < cols) return FP8_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(x) & (x_dt == FP8_F32 ? 3u : 1u)) return FP8_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const int32_t *bias = d_bias;
    if (!bias) {
        // FP8-AMAX.  Small contiguous tensors: one cluster holds the tensor in registers, one launch.
        if (!y_t && ld == cols && (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && (reinterpret_cast<uintptr_t>(y) & 7u) == 0 &&
            !g_no_small_cast) {
            cudaError_t se = launch_small_any(fmt, (int)x_dt, ctx, x, rows * cols, (int)conv, margin, d_amax_out,
                                              d_bias_out, y, st);
            if (se == cudaSuccess) return FP8_OK;
            cudaGetLastError();   // too large for the register-resident kernel (or the launch was refused)
        }
        // Otherwise amax + bias in one launch, the cast in a second.
        if (launch_amax_bias(ctx, x, (int)x_dt, rows, cols, ld, d_amax_out, d_bias_out, fmt, (int)conv, margin, st) !=
            cudaSuccess)
            return FP8_ERR_CUDA;
        bias = d_bias_out;
    }
    int delta = format_delta(fmt, (int)conv);
    // Delayed scaling: the bias is given AND the caller wants this tensor's own amax / bias (for the next step).
    const bool delayed = d_bias && d_amax_out && d_bias_out;
    if (delayed) {
        auto al16 = [](const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
        if (!y_t && ld == cols && al16(x) && al16(y)) {   // one pass: cast and amax together
            const int64_t n = rows * cols;
            cudaError_t pe;
#define FP8LIN_DELAYED(F, D) \
    pe = launch_predicted<F, D>(ctx, x, n, (int)conv, margin, d_amax_out, d_bias, d_bias_out, 0, y, st)
            if (fmt == FP8_E4) {
                if (x_dt == FP8_BF16) FP8LIN_DELAYED(FP8_E4, FP8_BF16);
                else if (x_dt == FP8_F16) FP8LIN_DELAYED(FP8_E4, FP8_F16);
                else FP8LIN_DELAYED(FP8_E4, FP8_F32);
            } else {
                if (x_dt == FP8_BF16) FP8LIN_DELAYED(FP8_E5, FP8_BF16);
                else if (x_dt == FP8_F16) FP8LIN_DELAYED(FP8_E5, FP8_F16);
                else FP8LIN_DELAYED(FP8_E5, FP8_F32);
            }
#undef FP8LIN_DELAYED
            return pe == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
        }
    }
    cudaError_t e = fmt == FP8_E4 ? launch_cast_dt<FP8_E4>((int)x_dt, ctx, x, rows, cols, ld, bias, delta, y, y_t, st)
                                  : launch_cast_dt<FP8_E5>((int)x_dt, ctx, x, rows, cols, ld, bias, delta, y, y_t, st);
    // other shapes: the cast above used d_bias (read before this launch overwrites d_bias_out, stream order)
    if (e == cudaSuccess && delayed)
        e = launch_amax_bias(ctx, x, (int)x_dt, rows, cols, ld, d_amax_out, d_bias_out, fmt, (int)conv, margin, st);
    return e == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

}  // namespace fp8lin

extern "C" {

fp8_status_t fp8_cast_e4(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                         const int32_t *d_bias, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                         int32_t *d_bias_out, uint8_t *y, uint8_t *y_t, void *stream)
{
    return fp8lin::cast_entry(FP8_E4, ctx, x, x_dt, rows, cols, ld, d_bias, conv, margin, d_amax_out, d_bias_out, y,
                              y_t, stream);
}

fp8_status_t fp8_cast_e5(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols, int64_t ld,
                         const int32_t *d_bias, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                         int32_t *d_bias_out, uint8_t *y, uint8_t *y_t, void *stream)
{
    return fp8lin::cast_entry(FP8_E5, ctx, x, x_dt, rows, cols, ld, d_bias, conv, margin, d_amax_out, d_bias_out, y,
                              y_t, stream);
}

fp8_status_t fp8_cast_predicted(fp8_ctx *ctx, fp8_format_t fmt, const void *x, fp8_dtype_t x_dt, int64_t rows,
                                int64_t cols, int64_t ld, fp8_conv_t conv, int32_t margin, float *d_amax_out,
                                int32_t *d_bias_inout, uint8_t *y, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !x || !y || !d_amax_out || !d_bias_inout) return FP8_ERR_NULL;
    if ((int)fmt < 0 || (int)fmt > 1 || (int)x_dt < 0 || (int)x_dt > 2 || (int)conv < 0 || (int)conv > 1)
        return FP8_ERR_DTYPE;
    if (rows <= 0 || cols <= 0 || ld < cols) return FP8_ERR_SHAPE;
    auto al16 = [](const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
    if (ld != cols || !al16(x) || !al16(y))   // outside the one-pass kernel's shape rules: the ordinary FP8-AMAX path
        return cast_entry((int)fmt, ctx, x, x_dt, rows, cols, ld, nullptr, conv, margin, d_amax_out, d_bias_inout, y,
                          nullptr, stream);
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t n = rows * cols;
    cudaError_t e;
#define FP8LIN_PRED(F, D) \
    e = launch_predicted<F, D>(ctx, x, n, (int)conv, margin, d_amax_out, d_bias_inout, d_bias_inout, 1, y, st)
    if (fmt == FP8_E4) {
        if (x_dt == FP8_BF16) FP8LIN_PRED(FP8_E4, FP8_BF16);
        else if (x_dt == FP8_F16) FP8LIN_PRED(FP8_E4, FP8_F16);
        else FP8LIN_PRED(FP8_E4, FP8_F32);
    } else {
        if (x_dt == FP8_BF16) FP8LIN_PRED(FP8_E5, FP8_BF16);
        else if (x_dt == FP8_F16) FP8LIN_PRED(FP8_E5, FP8_F16);
        else FP8LIN_PRED(FP8_E5, FP8_F32);
    }
#undef FP8LIN_PRED
    return e == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_prediction_stats(fp8_ctx *ctx, void *stream, unsigned *hits, unsigned *misses, int clear)
{
    if (!ctx || !hits || !misses) return FP8_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned host[2] = {0, 0};
    if (cudaMemcpyAsync(host, ctx->d_predict_stats, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return FP8_ERR_CUDA;
    if (clear && cudaMemsetAsync(ctx->d_predict_stats, 0, sizeof(host), st) != cudaSuccess) return FP8_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FP8_ERR_CUDA;
    *hits = host[0];
    *misses = host[1];
    return FP8_OK;
}

fp8_status_t fp8_range_stats(fp8_ctx *ctx, fp8_format_t fmt, const void *x, fp8_dtype_t x_dt, int64_t rows, int64_t cols,
                             int64_t ld, const int32_t *d_bias, fp8_conv_t conv, unsigned long long *d_counts,
                             void *stream)
{
    using namespace fp8lin;
    if (!ctx || !x || !d_bias || !d_counts) return FP8_ERR_NULL;
    if ((int)fmt < 0 || (int)fmt > 1 || (int)x_dt < 0 || (int)x_dt > 2 || (int)conv < 0 || (int)conv > 1)
        return FP8_ERR_DTYPE;
    if (rows <= 0 || cols <= 0 || ld < cols) return FP8_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(x) & (x_dt == FP8_F32 ? 3u : 1u)) || (reinterpret_cast<uintptr_t>(d_counts) & 7u))
        return FP8_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(d_counts, 0, 4 * sizeof(unsigned long long), st) != cudaSuccess) return FP8_ERR_CUDA;
    const int delta = format_delta((int)fmt, (int)conv);
    const int blocks = (int)(rows < ctx->sm_count * 8 ? rows : ctx->sm_count * 8);
#define FP8LIN_STATS(F, D) count_launch(), range_stats_kernel<F, D><<<blocks, 256, 0, st>>>(x, rows, cols, ld, d_bias, delta, d_counts)
    if (fmt == FP8_E4) {
        if (x_dt == FP8_BF16) FP8LIN_STATS(FP8_E4, FP8_BF16);
        else if (x_dt == FP8_F16) FP8LIN_STATS(FP8_E4, FP8_F16);
        else FP8LIN_STATS(FP8_E4, FP8_F32);
    } else {
        if (x_dt == FP8_BF16) FP8LIN_STATS(FP8_E5, FP8_BF16);
        else if (x_dt == FP8_F16) FP8LIN_STATS(FP8_E5, FP8_F16);
        else FP8LIN_STATS(FP8_E5, FP8_F32);
    }
#undef FP8LIN_STATS
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_ptq_weights(fp8_ctx *ctx, const void *w, fp8_dtype_t w_dt, int64_t N, int64_t K, int64_t ld,
                             fp8_conv_t conv, uint8_t *w8, uint8_t *w8_t, int32_t *d_bw, float *d_amax_w,
                             void *stream)
{
    return fp8lin::cast_entry(FP8_E4, ctx, w, w_dt, N, K, ld, nullptr, conv, 0, d_amax_w, d_bw, w8, w8_t, stream);
}

}  // extern "C"
