// FP8-AMAX as ONE launch: amax (Eq. 3), scaling bias, scale-and-cast (Eq. 1,
// Section 2.1) with both output layouts.
//
// The paper warns (Section 3) that computing the scale just in time costs a
// second round trip to memory unless the hardware has enough on-chip memory.
// A B200 has: 148 SMs x ~200 KB of shared memory hold 28 MB of bf16, and the
// L2 behind them holds the most recently read ~100 MB.  This kernel is
// persistent and cooperative (all CTAs resident):
//
//   phase 1  every CTA streams its contiguous run of 128x128 tiles through
//            shared memory with bulk tensor copies (one 32 KB copy per tile,
//            several in flight) and takes the packed integer max.  Its first
//            kStash tiles STAY in shared memory; the rest pass through a
//            two-slot ring.
//   barrier  one atomicMax and one arrival per CTA on a context slot; the wait
//            is bounded (sticky TIMEOUT flag, the kernel returns).
//   phase 2  every CTA derives the bias from the global amax and casts: first
//            the tiles still in shared memory (no memory read at all), then the
//            others newest-first, so that their second read is an L2 hit where
//            the tensor allows.  Outputs leave in 128-byte rows, the transposed
//            copy through the rotated staging tile of the two-launch kernel.
//
// Algorithmic traffic: 2 B read + 1 B per layout written per element.
#include <algorithm>

#include "cast_common.cuh"
#include "ptx.cuh"

namespace fp8lin {

constexpr int kFusedThreads = 512;
constexpr int kFT = 128;                         // tile edge
constexpr int kFTileBytes = kFT * kFT * 2;       // 32 KB of bf16
constexpr int kFSlots = 6;                       // shared-memory tile slots
constexpr int kStash = kFSlots - 2;              // tiles that stay resident; the last two slots form the ring
constexpr int kFStageBytes = kFT * kFT;          // transposed staging, 16 KB
constexpr int kFusedSmem = kFSlots * kFTileBytes + kFStageBytes + 64 + 128;

struct FusedParams {
    int64_t rows, cols;
    int tiles_c, num_tiles;
    int fmt, conv, margin, delta;
    unsigned *slot;        // {running max, arrivals, departures}
    float *d_amax;
    int32_t *d_bias;
    unsigned *d_status;
    uint8_t *y, *y_t;
};

__device__ __forceinline__ int slot_of(int i) { return i < kStash ? i : kStash + ((i - kStash) & 1); }

template <int FMT>
__device__ __forceinline__ void convert_tile(const uint8_t *tile, uint32_t (*stage)[kFT / 4], const FusedParams &p,
                                             int64_t r0, int64_t c0, Pow2Pair sc, bool &sat, int warp, int lane)
{
    // 32 x 32 blocks of 4 rows x 4 columns; 16 warps take two block-rows each, a lane one block-column
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int rg = warp + 16 * it;
        uint32_t rw[4], cw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint2 v = *reinterpret_cast<const uint2 *>(tile + (4 * rg + i) * (kFT * 2) + 8 * lane);
            rw[i] = cast4<FMT, true>(v.x, v.y, sc, sat);
        }
        if (p.y) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                *reinterpret_cast<uint32_t *>(p.y + (r0 + 4 * rg + i) * p.cols + c0 + 4 * lane) = rw[i];
        }
        if (p.y_t) {
            transpose4x4(rw, cw);
#pragma unroll
            for (int j = 0; j < 4; ++j) stage[4 * lane + j][(rg + lane) & 31] = cw[j];
        }
    }
    if (p.y_t) {
        __syncthreads();
#pragma unroll 4
        for (int cc = warp; cc < kFT; cc += 16) {
            const uint32_t w = stage[cc][(lane + (cc >> 2)) & 31];
            *reinterpret_cast<uint32_t *>(p.y_t + (c0 + cc) * p.rows + r0 + 4 * lane) = w;
        }
        __syncthreads();  // the staging tile is free again
    }
}

template <int FMT>
__global__ void __launch_bounds__(kFusedThreads, 1)
cast_fused_kernel(const __grid_constant__ CUtensorMap map_x, const FusedParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    uint8_t *tiles = smem;
    uint32_t(*stage)[kFT / 4] = reinterpret_cast<uint32_t(*)[kFT / 4]>(smem + kFSlots * kFTileBytes);
    const uint32_t bar0 = smem_u32(smem + kFSlots * kFTileBytes + kFStageBytes);
    __shared__ uint32_t warp_max[kFusedThreads / 32];
    __shared__ uint32_t bcast[2];
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // contiguous run of tiles for this CTA
    const int base = p.num_tiles / gridDim.x, extra = p.num_tiles % gridDim.x;
    const int first = blockIdx.x * base + min((int)blockIdx.x, extra);
    const int n_my = base + ((int)blockIdx.x < extra ? 1 : 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFSlots; ++s) mbar_init(bar0 + 8u * s, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    auto issue = [&](int i) {  // thread 0 only: start the copy of this CTA's i-th tile into its slot
        const int t = first + i;
        const int s = slot_of(i);
        mbar_expect_tx(bar0 + 8u * s, kFTileBytes);
        tma_load_2d(smem_u32(tiles + s * kFTileBytes), &map_x, bar0 + 8u * s, (t % p.tiles_c) * kFT, (t / p.tiles_c) * kFT);
    };
    uint32_t phase_bits = 0;  // one parity bit per slot, tracked identically by every thread
    auto wait_slot = [&](int s) -> bool {
        const bool ok = mbar_wait(bar0 + 8u * s, (phase_bits >> s) & 1u, &abort_flag, p.d_status);
        phase_bits ^= 1u << s;
        return ok;
    };

    // ------------------------------- phase 1: amax -------------------------------
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
        for (int i = 0; i < min(n_my, kFSlots); ++i) issue(i);
    }
    uint32_t acc = 0;
    bool alive = true;
    for (int i = 0; i < n_my && alive; ++i) {
        const int s = slot_of(i);
        alive = __syncthreads_and(wait_slot(s) ? 1 : 0) != 0;  // the whole CTA goes on, or none of it
        if (!alive) break;
        const uint4 *src = reinterpret_cast<const uint4 *>(tiles + s * kFTileBytes);
#pragma unroll
        for (int j = 0; j < kFTileBytes / 16 / kFusedThreads; ++j) {
            const uint4 v = src[threadIdx.x + j * kFusedThreads];
            acc = __vmaxu2(acc, v.x & 0x7FFF7FFFu);
            acc = __vmaxu2(acc, v.y & 0x7FFF7FFFu);
            acc = __vmaxu2(acc, v.z & 0x7FFF7FFFu);
            acc = __vmaxu2(acc, v.w & 0x7FFF7FFFu);
        }
        // a ring slot is refilled two tiles ahead, once every thread has read it; the last two ring tiles
        // stay where they are for phase 2
        if (i >= kStash && i + 2 < n_my) {
            __syncthreads();
            if (threadIdx.x == 0) issue(i + 2);
        }
    }
    uint32_t m = max(acc & 0xFFFFu, acc >> 16);
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (lane == 0) warp_max[warp] = m;
    __syncthreads();

    // ------------------------------- grid barrier -------------------------------
    if (threadIdx.x == 0) {
        for (int i = 1; i < kFusedThreads / 32; ++i) m = max(m, warp_max[i]);
        atomicMax(&p.slot[0], m);
        __threadfence();
        atomicAdd(&p.slot[1], 1u);
        const unsigned long long t0 = global_timer_ns();
        bool ok = abort_flag == 0;
        while (ok && *reinterpret_cast<volatile unsigned *>(&p.slot[1]) < gridDim.x) {
            __nanosleep(64);
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                atomicOr(p.d_status, FP8_FLAG_TIMEOUT);
                ok = false;
            }
        }
        __threadfence();
        const uint32_t total = *reinterpret_cast<volatile unsigned *>(&p.slot[0]);
        bcast[0] = total;
        bcast[1] = ok ? 1u : 0u;
        // the last CTA to have read the result leaves the slot zeroed for the next call
        if (atomicAdd(&p.slot[2], 1u) + 1u == gridDim.x) {
            p.slot[0] = 0u;
            p.slot[1] = 0u;
            p.slot[2] = 0u;
        }
    }
    __syncthreads();
    if (bcast[1] == 0u) {  // a wait expired: outputs are invalid; give copies already issued time to land
        __nanosleep(20000);
        return;
    }

    const uint32_t fbits = bcast[0] << 16;
    unsigned flags = 0;
    const int bias = bias_from_amax_bits(fbits, p.fmt, p.conv, p.margin, &flags);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *p.d_amax = __uint_as_float(fbits);
        *p.d_bias = bias;
        if (flags) atomicOr(p.d_status, flags);
    }
    const Pow2Pair sc = make_pow2_pair(bias + p.delta);
    bool sat = false;

    // ------------------------------- phase 2: cast -------------------------------
    // resident tiles: the stash, then the (up to) two newest ring tiles
    const int n_stash = min(n_my, kStash);
    for (int i = 0; i < n_stash; ++i) {
        const int t = first + i;
        convert_tile<FMT>(tiles + slot_of(i) * kFTileBytes, stage, p, (int64_t)(t / p.tiles_c) * kFT,
                          (int64_t)(t % p.tiles_c) * kFT, sc, sat, warp, lane);
    }
    const int newest = n_my - 1;
    const int resident_from = max(kStash, n_my - 2);  // ring tiles still in shared memory
    // start re-loading the older ring tiles, newest first, as slots become free
    int next_reload = resident_from - 1;               // next tile index to fetch again (descending)
    for (int i = newest; i >= kStash; --i) {
        const int s = slot_of(i);
        if (i < resident_from) {
            if (__syncthreads_and(wait_slot(s) ? 1 : 0) == 0) break;
        }
        const int t = first + i;
        convert_tile<FMT>(tiles + s * kFTileBytes, stage, p, (int64_t)(t / p.tiles_c) * kFT,
                          (int64_t)(t % p.tiles_c) * kFT, sc, sat, warp, lane);
        // this slot is free now: fetch the next older tile that maps to it
        __syncthreads();
        if (next_reload >= kStash) {
            if (threadIdx.x == 0) issue(next_reload);
            --next_reload;
        }
    }
    if (__syncthreads_or(sat) && threadIdx.x == 0) atomicOr(p.d_status, FP8_FLAG_SATURATED);
}

static bool g_fused_ready = false;
static bool g_fused_off = false;

cudaError_t launch_cast_fused(fp8_ctx *ctx, int fmt, const void *x, int64_t rows, int64_t cols, int64_t ld, int conv,
                              int margin, float *d_amax_out, int32_t *d_bias_out, uint8_t *y, uint8_t *y_t,
                              cudaStream_t stream)
{
    if (!g_fused_ready) {
        if (kFusedSmem > ctx->max_smem_optin) return cudaErrorNotSupported;
        cudaError_t e = cudaFuncSetAttribute(cast_fused_kernel<FP8_E4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kFusedSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(cast_fused_kernel<FP8_E5>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem);
        if (e != cudaSuccess) return e;
        const char *env = getenv("FP8LIN_FUSED_CAST");  // opt-in: slower than the two-launch path as it stands
        g_fused_off = !(env && env[0] == '1');
        g_fused_ready = true;
    }
    auto al = [](const void *q, unsigned a) { return (reinterpret_cast<uintptr_t>(q) & (a - 1)) == 0; };
    // shape rules of this kernel: whole 128x128 tiles, 16-byte aligned rows, at least a few tiles per SM's worth of work
    if (g_fused_off || (rows % kFT) || (cols % kFT) || (ld % 8) || !al(x, 16) || (y && !al(y, 4)) || (y_t && !al(y_t, 4)))
        return cudaErrorNotSupported;
    const int64_t tiles = (rows / kFT) * (cols / kFT);
    if (tiles > 0x7FFFFFFF || cols > 0x7FFFFFFF || rows > 0x7FFFFFFF) return cudaErrorNotSupported;

    CUtensorMap map_x;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)(ld * 2)};
    cuuint32_t box[2] = {kFT, kFT};
    cuuint32_t estr[2] = {1, 1};
    if (ctx->encode_tiled(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void *>(x), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorNotSupported;

    FusedParams p;
    p.rows = rows; p.cols = cols;
    p.tiles_c = (int)(cols / kFT);
    p.num_tiles = (int)tiles;
    p.fmt = fmt; p.conv = conv; p.margin = margin; p.delta = format_delta(fmt, conv);
    p.slot = take_slot(ctx);
    p.d_amax = d_amax_out; p.d_bias = d_bias_out; p.d_status = ctx->d_status;
    p.y = y; p.y_t = y_t;
    int grid = (int)std::min<int64_t>(tiles, ctx->sm_count);
    void *args[2] = {&map_x, &p};
    const void *fn = fmt == FP8_E4 ? (const void *)cast_fused_kernel<FP8_E4> : (const void *)cast_fused_kernel<FP8_E5>;
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kFusedThreads), args, kFusedSmem, stream);
}

}  // namespace fp8lin
