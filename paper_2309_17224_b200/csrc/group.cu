// Grouped FP8-AMAX quantisation: amax -> bias -> scale-and-cast (Eq. 3, Eq. 1, Section 2.1 / 2.2) of several
// tensors in two launches instead of two per tensor.  The same kernels, on a group of one, serve every contiguous
// single-tensor call (fp8_amax, fp8_cast_e4 / _e5, fp8_cast_predicted, delayed scaling).
//
// The tensors a step quantises are tens to hundreds of megabytes each; launched one by one, every kernel pays its
// own ramp-up and its own thin last wave, which at these sizes is 10-40 % of its run time.  Here the tensors of a
// group are cut into chunks of a few thousand elements, the chunks of all tensors are numbered in one sequence and a
// persistent grid walks that sequence with a grid stride, so the whole group has one ramp and one tail.  Each
// tensor keeps its own reduction slot: a block notes its maximum of a tensor when it moves on to the next one, folds
// all its notes into the slots at the end (one thread per tensor), adds the number of chunks it did, and the block
// that completes a tensor's count publishes that tensor's amax and bias.
//
// Two modes, both bit-identical to fp8_cast_e4 / fp8_cast_e5 with d_bias = NULL per tensor:
//   just in time   group_kernel<kAmax> over all tensors, then group_kernel<kCast> (a programmatic dependent) over
//                  all tensors back to front: 2 B read + (2 B read + 1 B written) per 16-bit element.
//   predicted      group_kernel<kBoth> casts every tensor with the bias found in its bias word (a guess, normally
//                  the previous step's) while it takes the amax; the block that completes a tensor derives the
//                  true bias and raises that tensor's redo flag if the guess was wrong; the second launch
//                  (kCast, gated per tensor) redoes only those tensors.  2 B read + 1 B written per element when
//                  every guess holds.
#include "cast_common.cuh"

namespace fp8lin {

constexpr int kGroupMax = FP8_GROUP_MAX;
// Measured on the twelve tensors of a Llama-2-7B step (1.5 GB of bf16): four output vectors per thread and chunk
// (eight 16-byte loads in flight per thread), three resident blocks per SM for the read-only pass and two for the
// passes that also write, streaming stores: amax 7.0 TB/s, cast 6.7 TB/s, one pass 6.3 TB/s.  More blocks per SM
// cost the writing passes up to a third of their bandwidth (5 per SM: 5.8 TB/s).
// (FP32 inputs bring twice the bytes per output vector: two output vectors per thread keep them in registers.)
#ifndef FP8LIN_GROUP_UNROLL
#define FP8LIN_GROUP_UNROLL 4
#endif
#ifndef FP8LIN_GROUP_AMAX_BLOCKS
#define FP8LIN_GROUP_AMAX_BLOCKS 3
#endif
#ifndef FP8LIN_GROUP_CAST_BLOCKS
#define FP8LIN_GROUP_CAST_BLOCKS 2
#endif
__host__ __device__ constexpr int group_unroll(int dt) { return dt == FP8_F32 ? 2 : FP8LIN_GROUP_UNROLL; }   // output vectors per thread and chunk
__host__ __device__ constexpr int group_blocks_per_sm(int mode) { return mode == 0 ? FP8LIN_GROUP_AMAX_BLOCKS : FP8LIN_GROUP_CAST_BLOCKS; }
__host__ __device__ constexpr int group_chunk_out(int dt) { return group_unroll(dt) * kCastThreads; }   // output vectors per chunk

struct GroupItem {
    const uint4 *x;
    uint4 *y;
    int64_t n;             // elements
    int64_t first_chunk;   // number of chunks of the items before this one
    int64_t chunks;        // >= 1
    int dt, fmt, margin, delta;
    unsigned *slot;        // {running max, chunks done, saturation seen, redo}
    float *d_amax;
    const int32_t *d_bias_in;   // the bias a casting pass applies (a guess, in the one-pass mode)
    int32_t *d_bias;            // where the amax passes write the Eq. 3 bias (may be NULL: amax only)
};

struct GroupParams {
    int count, conv;
    int verify;            // one-pass mode: the given bias is a guess to be checked (else it is simply the bias to use)
    int64_t total_chunks;
    unsigned *d_status, *d_stats;
    GroupItem it[kGroupMax];
};

enum { kAmax = 0, kCast = 1, kBoth = 2 };

__device__ __forceinline__ uint32_t fold_any(int dt, uint32_t acc, uint32_t w)
{
    return dt == FP8_F32 ? max(acc, w & 0x7FFFFFFFu) : __vmaxu2(acc, w & 0x7FFF7FFFu);
}

// One chunk of one tensor: thread t owns output vectors c * chunk + t + u * 256, u < group_unroll(DT).
template <int MODE, int FMT, int DT, bool TWO_STEP>
__device__ __forceinline__ void chunk_body(const uint4 *__restrict__ gx, uint4 *__restrict__ gy, int64_t n, int64_t c,
                                           Pow2Pair p, uint32_t &acc, bool &sat)
{
    constexpr int kIn = InType<DT>::kBytes;   // input vectors per output vector
    constexpr int kW = InType<DT>::kWords4;
    constexpr int kUnroll = group_unroll(DT);
    constexpr int kChunkOut = group_chunk_out(DT);
    const int64_t nout = n / 16;
    int64_t idx[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) idx[u] = c * kChunkOut + threadIdx.x + u * kCastThreads;
    uint4 v[kUnroll][kIn];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
        if (idx[u] < nout) {
#pragma unroll
            for (int j = 0; j < kIn; ++j)
                v[u][j] = MODE == kAmax ? __ldg(gx + kIn * idx[u] + j) : __ldcs(gx + kIn * idx[u] + j);
        }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
        if (idx[u] < nout) {
            const uint32_t *w = reinterpret_cast<const uint32_t *>(&v[u][0]);
            if (MODE != kCast) {
#pragma unroll
                for (int j = 0; j < 4 * kIn; ++j) acc = fold_any(DT, acc, w[j]);
            }
            if (MODE != kAmax) {
                uint4 o;
                o.x = cast4w<FMT, DT, TWO_STEP>(w + 0 * kW, p, sat);
                o.y = cast4w<FMT, DT, TWO_STEP>(w + 1 * kW, p, sat);
                o.z = cast4w<FMT, DT, TWO_STEP>(w + 2 * kW, p, sat);
                o.w = cast4w<FMT, DT, TWO_STEP>(w + 3 * kW, p, sat);
                __stcs(gy + idx[u], o);   // the bytes are read next by a matmul, long after this pass
            }
        }
    // the elements past the last whole output vector belong to the tensor's first chunk
    const int ntail = (int)(n - nout * 16);
    if (c == 0 && (int)threadIdx.x < ntail) {
        const int64_t i = nout * 16 + threadIdx.x;
        if (MODE != kCast) {
            if (DT == FP8_F32) acc = max(acc, reinterpret_cast<const uint32_t *>(gx)[i] & 0x7FFFFFFFu);
            else acc = __vmaxu2(acc, (uint32_t)reinterpret_cast<const uint16_t *>(gx)[i] & 0x7FFFu);
        }
        if (MODE != kAmax) reinterpret_cast<uint8_t *>(gy)[i] = cast1<FMT, DT, true>(gx, i, p, sat);
    }
}

// This block's chunks of one tensor: `iters` chunks starting at tensor-local chunk `c`, `step` apart.  The scaling
// always takes the two-factor form (the second factor is 1 unless the shift leaves [-126, 127]): one multiply more
// per element, far below what the memory pipe leaves idle, and half as many code paths.
template <int MODE, int DT>
__device__ __forceinline__ void item_loop(const GroupItem &g, int64_t c, int64_t step, int64_t iters, Pow2Pair p,
                                          uint32_t &acc, bool &sat)
{
    if (MODE == kAmax || g.fmt == FP8_E4) {
        for (int64_t k = 0; k < iters; ++k, c += step) chunk_body<MODE, FP8_E4, DT, true>(g.x, g.y, g.n, c, p, acc, sat);
    } else {
        for (int64_t k = 0; k < iters; ++k, c += step) chunk_body<MODE, FP8_E5, DT, true>(g.x, g.y, g.n, c, p, acc, sat);
    }
}

// What a block found in the tensors it walked, kept in shared memory until the end of the kernel: the block's
// maximum, how many chunks it did, whether a value clipped, the guess it cast with.
struct BlockNotes {
    uint32_t max_key[kGroupMax];
    unsigned done[kGroupMax];
    unsigned sat[kGroupMax];
    int guess[kGroupMax];
};

// A block leaves tensor `item` after `done` chunks: reduce its maximum across the block and note it.
__device__ __forceinline__ void note_item(BlockNotes &notes, int item, int dt, uint32_t acc, bool sat, unsigned done, int guess)
{
    __shared__ uint32_t warp_max[kCastThreads / 32];
    uint32_t m = dt == FP8_F32 ? acc : max(acc & 0xFFFFu, acc >> 16);
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    const int any_sat = __syncthreads_or(sat);
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 1; i < kCastThreads / 32; ++i) m = max(m, warp_max[i]);
        notes.max_key[item] = m;
        notes.done[item] = done;
        notes.sat[item] = any_sat ? 1u : 0u;
        notes.guess[item] = guess;
    }
    __syncthreads();   // warp_max is reused by the next tensor
}

// End of the kernel: one thread per tensor folds the block's note into the tensor's slot (all tensors at once, so
// the block pays one round trip to the atomics and not one per tensor); the thread that completes a tensor's chunk
// count publishes its amax and bias and, in the predicted mode, the verdict on the guess.
template <int MODE>
__device__ __forceinline__ void publish_item(const GroupItem &g, const BlockNotes &notes, int item, int conv, int verify,
                                             unsigned *d_status, unsigned *d_stats)
{
    const unsigned done = notes.done[item];
    if (done == 0u) return;
    atomicMax(&g.slot[0], notes.max_key[item]);
    if (MODE == kBoth && notes.sat[item]) atomicOr(&g.slot[2], 1u);
    __threadfence();
    if (atomicAdd(&g.slot[1], done) + done != (unsigned)g.chunks) return;
    __threadfence();
    const uint32_t total = atomicExch(&g.slot[0], 0u);
    const unsigned was_sat = atomicExch(&g.slot[2], 0u);
    g.slot[1] = 0u;
    uint32_t fbits;
    if (g.dt == FP8_F32) fbits = total;
    else if (g.dt == FP8_BF16) fbits = total << 16;
    else { float f; asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"((uint16_t)total)); fbits = __float_as_uint(f); }
    *g.d_amax = __uint_as_float(fbits);
    unsigned flags = 0;
    const int b = bias_from_amax_bits(fbits, g.fmt, conv, g.margin, &flags);
    if (g.d_bias == nullptr) return;   // amax alone was asked for: no bias, no flags
    *g.d_bias = b;
    if (MODE == kBoth) {
        const bool hit = b == notes.guess[item] || !verify;
        g.slot[3] = hit ? 0u : 1u;   // read by the gated second launch
        if (verify) atomicAdd(&d_stats[hit ? 0 : 1], 1u);
        if (hit && was_sat) flags |= FP8_FLAG_SATURATED;   // clipping under a wrong guess says nothing
    }
    if (flags) atomicOr(d_status, flags);
}

// Item `i` of the parameter block.  Kernel parameters cannot be indexed by a run-time value without the compiler
// copying the whole block into every thread's local memory; sixteen compile-time indices can.
__device__ __forceinline__ GroupItem get_item(const GroupParams &gp, int i)
{
    static_assert(kGroupMax == 16, "one case per item");
    switch (i) {
#define FP8LIN_ITEM(k) case k: return gp.it[k];
        FP8LIN_ITEM(0) FP8LIN_ITEM(1) FP8LIN_ITEM(2) FP8LIN_ITEM(3) FP8LIN_ITEM(4) FP8LIN_ITEM(5) FP8LIN_ITEM(6) FP8LIN_ITEM(7)
        FP8LIN_ITEM(8) FP8LIN_ITEM(9) FP8LIN_ITEM(10) FP8LIN_ITEM(11) FP8LIN_ITEM(12) FP8LIN_ITEM(13) FP8LIN_ITEM(14)
#undef FP8LIN_ITEM
    default: return gp.it[15];
    }
}

// gate != 0 (kCast only): cast only the tensors whose redo flag is raised.
//
// The chunks of all tensors are numbered in one sequence; block b takes numbers b, b + grid, b + 2 grid, ...  The
// amax passes count from the front of the first tensor; the cast pass counts from the back of the last one, so that
// what the amax pass read last (and may still be in L2) is read first.
template <int MODE, int DT>
__global__ void __launch_bounds__(kCastThreads, group_blocks_per_sm(MODE)) group_kernel(const __grid_constant__ GroupParams gp, int gate)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (MODE == kCast) asm volatile("griddepcontrol.wait;" ::: "memory");   // biases / redo flags of the launch before
    const int64_t grid = gridDim.x, b = blockIdx.x;
    bool any_sat = false;
    __shared__ BlockNotes notes;
    // the bias every tensor is cast with and, for the gated pass, its redo flag: fetched by one thread per tensor at
    // once (a block that fetched them tensor by tensor would pay one trip to L2 per tensor before touching its data)
    __shared__ int given_bias[kGroupMax];
    __shared__ unsigned redo[kGroupMax];
    if ((int)threadIdx.x < gp.count) {
        const GroupItem g = get_item(gp, threadIdx.x);
        notes.done[threadIdx.x] = 0u;
        if (MODE != kAmax) given_bias[threadIdx.x] = *reinterpret_cast<const volatile int32_t *>(g.d_bias_in);
        if (MODE == kCast) redo[threadIdx.x] = gate ? *reinterpret_cast<const volatile unsigned *>(&g.slot[3]) : 1u;
    }
    __syncthreads();
    for (int n = 0; n < gp.count; ++n) {
        const int item = MODE == kCast ? gp.count - 1 - n : n;
        if (MODE == kCast && redo[item] == 0u) continue;
        const GroupItem g = get_item(gp, item);
        // sequence numbers of this tensor's chunks: [lo, lo + chunks); number lo + j is tensor-local chunk j in the
        // forward passes and chunk (chunks - 1 - j) in the backward pass
        const int64_t lo = MODE == kCast ? gp.total_chunks - g.first_chunk - g.chunks : g.first_chunk;
        const int64_t k0 = lo > b ? (lo - b + grid - 1) / grid : 0;   // first k with b + k grid >= lo
        const int64_t j0 = b + k0 * grid - lo;
        const int64_t iters = j0 < g.chunks ? (g.chunks - j0 + grid - 1) / grid : 0;
        if (iters == 0) continue;
        int guess = 0;
        Pow2Pair p = make_pow2_pair(0);
        if (MODE != kAmax) {
            guess = given_bias[item];
            p = make_pow2_pair(guess + g.delta);
        }
        uint32_t acc = 0;
        bool sat = false;
        if (MODE == kCast) item_loop<MODE, DT>(g, g.chunks - 1 - j0, -grid, iters, p, acc, sat);
        else item_loop<MODE, DT>(g, j0, grid, iters, p, acc, sat);
        if (MODE == kCast) any_sat = any_sat || sat;
        else note_item(notes, item, g.dt, acc, sat, (unsigned)iters, guess);
    }
    if (MODE == kCast) {
        if (__syncthreads_or(any_sat) && threadIdx.x == 0) atomicOr(gp.d_status, (unsigned)FP8_FLAG_SATURATED);
    } else if ((int)threadIdx.x < gp.count) {   // note_item ended on a barrier: the notes are complete
        publish_item<MODE>(get_item(gp, threadIdx.x), notes, threadIdx.x, gp.conv, gp.verify, gp.d_status, gp.d_stats);
    }
}

// One pass over up to kGroupMax tensors of one input type.  `first`: kAmax, kBoth or kCast launched as an ordinary
// kernel; a kCast pass behind another pass of the same call is launched as its programmatic dependent.
static cudaError_t launch_pass(fp8_ctx *ctx, const GroupParams &gp, int dt, int mode, int gate, bool dependent, cudaStream_t st)
{
    const int64_t cap = (int64_t)ctx->sm_count * group_blocks_per_sm(mode);   // the blocks resident at once (launch bounds)
    const unsigned blocks = (unsigned)(gp.total_chunks < cap ? gp.total_chunks : cap);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(kCastThreads);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    count_launch();
#define FP8LIN_PASS(M) \
    (dt == FP8_BF16  ? cudaLaunchKernelEx(&cfg, group_kernel<M, FP8_BF16>, gp, gate) \
     : dt == FP8_F16 ? cudaLaunchKernelEx(&cfg, group_kernel<M, FP8_F16>, gp, gate) \
                     : cudaLaunchKernelEx(&cfg, group_kernel<M, FP8_F32>, gp, gate))
    if (mode == kAmax) return FP8LIN_PASS(kAmax);
    if (mode == kBoth) return FP8LIN_PASS(kBoth);
    return FP8LIN_PASS(kCast);
#undef FP8LIN_PASS
}

static void add_item(fp8_ctx *ctx, GroupParams &gp, const void *x, void *y, int64_t n, int dt, int fmt, int margin, int conv,
                     float *d_amax, const int32_t *d_bias_in, int32_t *d_bias_out)
{
    GroupItem &g = gp.it[gp.count++];
    g.x = reinterpret_cast<const uint4 *>(x);
    g.y = reinterpret_cast<uint4 *>(y);
    g.n = n;
    g.first_chunk = gp.total_chunks;
    g.chunks = (n / 16 + group_chunk_out(dt) - 1) / group_chunk_out(dt);
    if (g.chunks < 1) g.chunks = 1;
    gp.total_chunks += g.chunks;
    g.dt = dt;
    g.fmt = fmt;
    g.margin = margin;
    g.delta = format_delta(fmt, conv);
    g.slot = take_slot(ctx);
    g.d_amax = d_amax;
    g.d_bias_in = d_bias_in;
    g.d_bias = d_bias_out;
}

static GroupParams empty_group(fp8_ctx *ctx, int conv, int verify)
{
    GroupParams gp;
    gp.count = 0;
    gp.conv = conv;
    gp.verify = verify;
    gp.total_chunks = 0;
    gp.d_status = ctx->d_status;
    gp.d_stats = ctx->d_predict_stats;
    return gp;
}

// The same kernels for ONE contiguous, 16-byte aligned tensor (the single-tensor entry points route here).
cudaError_t launch_amax_flat(fp8_ctx *ctx, const void *x, int dt, int64_t n, float *d_amax, int32_t *d_bias, int fmt,
                             int conv, int margin, cudaStream_t st)
{
    GroupParams gp = empty_group(ctx, conv, 0);
    add_item(ctx, gp, x, nullptr, n, dt, fmt, margin, conv, d_amax, d_bias, d_bias);
    return launch_pass(ctx, gp, dt, kAmax, 0, false, st);
}

cudaError_t launch_cast_flat(fp8_ctx *ctx, const void *x, int dt, int64_t n, const int32_t *d_bias, int fmt, int delta,
                             uint8_t *y, cudaStream_t st)
{
    GroupParams gp = empty_group(ctx, FP8_CONV_PAPER, 0);
    add_item(ctx, gp, x, y, n, dt, fmt, 0, FP8_CONV_PAPER, nullptr, d_bias, nullptr);
    gp.it[0].delta = delta;   // the format shift comes from the caller; a cast pass needs nothing else of the convention
    return launch_pass(ctx, gp, dt, kCast, 0, true, st);   // may follow an amax pass as its programmatic dependent
}

cudaError_t launch_one_pass_flat(fp8_ctx *ctx, const void *x, int dt, int64_t n, int fmt, int conv, int margin,
                                 float *d_amax, const int32_t *d_bias_in, int32_t *d_bias_out, int verify, uint8_t *y,
                                 cudaStream_t st)
{
    GroupParams gp = empty_group(ctx, conv, verify);
    add_item(ctx, gp, x, y, n, dt, fmt, margin, conv, d_amax, d_bias_in, d_bias_out);
    cudaError_t e = launch_pass(ctx, gp, dt, kBoth, 0, false, st);
    if (e != cudaSuccess || !verify) return e;
    gp.it[0].d_bias_in = d_bias_out;   // the redo, if any, uses the bias the first pass published
    return launch_pass(ctx, gp, dt, kCast, 1, true, st);
}

static bool group_shape_ok(const fp8_group_item_t &t)
{
    auto al16 = [](const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
    return t.ld == t.cols && al16(t.x) && al16(t.y);   // a NULL y (amax only) passes
}

}  // namespace fp8lin

extern "C" {

fp8_status_t fp8_cast_group(fp8_ctx *ctx, const fp8_group_item_t *items, int32_t count, fp8_conv_t conv,
                            fp8_group_mode_t mode, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !items) return FP8_ERR_NULL;
    if (count <= 0) return FP8_ERR_SHAPE;
    if ((int)conv < 0 || (int)conv > 1 || (int)mode < 0 || (int)mode > 3) return FP8_ERR_DTYPE;
    const bool predicted = mode == FP8_GROUP_PREDICTED;
    const bool want_amax = mode != FP8_GROUP_CAST_ONLY, want_cast = mode != FP8_GROUP_AMAX_ONLY;
    for (int i = 0; i < count; ++i) {
        const fp8_group_item_t &t = items[i];
        if (!t.x || (want_cast && !t.y) || (want_amax && !t.d_amax) || !t.d_bias) return FP8_ERR_NULL;
        if ((int)t.fmt < 0 || (int)t.fmt > 1 || (int)t.x_dt < 0 || (int)t.x_dt > 2) return FP8_ERR_DTYPE;
        if (t.rows <= 0 || t.cols <= 0 || t.ld < t.cols) return FP8_ERR_SHAPE;
        if (reinterpret_cast<uintptr_t>(t.x) & (t.x_dt == FP8_F32 ? 3u : 1u)) return FP8_ERR_ALIGN;
    }
    cudaStream_t st = (cudaStream_t)stream;
    int i = 0;
    while (i < count) {
        // tensors outside the grouped kernels' shape rules go through the single-tensor entry points
        if (!group_shape_ok(items[i])) {
            const fp8_group_item_t &t = items[i];
            fp8_status_t s;
            if (predicted) {
                s = fp8_cast_predicted(ctx, t.fmt, t.x, t.x_dt, t.rows, t.cols, t.ld, conv, t.margin, t.d_amax, t.d_bias, t.y,
                                       stream);
            } else if (mode == FP8_GROUP_AMAX_ONLY) {
                s = launch_amax_bias(ctx, t.x, (int)t.x_dt, t.rows, t.cols, t.ld, t.d_amax, t.d_bias, (int)t.fmt, (int)conv,
                                     t.margin, st) == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
            } else {
                const int32_t *given = mode == FP8_GROUP_CAST_ONLY ? t.d_bias : nullptr;
                float *ao = given ? nullptr : t.d_amax;
                int32_t *bo = given ? nullptr : t.d_bias;
                s = t.fmt == FP8_E4 ? fp8_cast_e4(ctx, t.x, t.x_dt, t.rows, t.cols, t.ld, given, conv, t.margin, ao, bo, t.y,
                                                  nullptr, stream)
                                    : fp8_cast_e5(ctx, t.x, t.x_dt, t.rows, t.cols, t.ld, given, conv, t.margin, ao, bo, t.y,
                                                  nullptr, stream);
            }
            if (s != FP8_OK) return s;
            ++i;
            continue;
        }
        GroupParams gp = empty_group(ctx, (int)conv, predicted ? 1 : 0);
        const int dt = (int)items[i].x_dt;   // one input type per pair of launches
        while (i < count && gp.count < kGroupMax && group_shape_ok(items[i]) && (int)items[i].x_dt == dt) {
            const fp8_group_item_t &t = items[i];
            if ((t.rows * t.cols / 16 + group_chunk_out(dt) - 1) / group_chunk_out(dt) > 0x7FFFFFFF) return FP8_ERR_SHAPE;
            add_item(ctx, gp, t.x, t.y, t.rows * t.cols, dt, (int)t.fmt, t.margin, (int)conv, t.d_amax, t.d_bias, t.d_bias);
            ++i;
        }
        if (want_amax && launch_pass(ctx, gp, dt, predicted ? kBoth : kAmax, 0, false, st) != cudaSuccess) return FP8_ERR_CUDA;
        if (want_cast && launch_pass(ctx, gp, dt, kCast, predicted ? 1 : 0, true, st) != cudaSuccess) return FP8_ERR_CUDA;
    }
    return FP8_OK;
}

}  // extern "C"
