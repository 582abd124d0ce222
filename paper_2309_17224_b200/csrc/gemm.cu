// FP8 matmuls with the unscale folded into the epilogue (Fig. 3b, Eq. 2 for the
// forward pass; Section 2.2 for the two backward matmuls).
//
// D[M,N] = A * B^T over a contraction of length K, computed by one of two
// persistent, warp-specialised kernels that share every building block:
//
//   gemm_pair_kernel  (M > 128)  two CTAs of a cluster own one 256x256 tile;
//                     tcgen05.mma.cta_group::2, six stages of 32 KB per CTA.
//   gemm_kernel       (M <= 128)  one CTA owns a 128x256 tile,
//                     four stages of 48 KB, optional split of the contraction
//                     (partial sums in an FP32 workspace, splitk_finalize_kernel
//                     launched behind it as a programmatic dependent).
//   decode_kernel     (M <= 128, contraction-major operands, plain epilogue)
//                     gemm_kernel with tile width, stage count and split chosen
//                     per launch, a tile's contraction shared by a cluster, and
//                     optionally the activation quantised by the same launch.
//
// Roles in all of them:
//   warp 0, one lane   TMA producer: 128-byte-swizzled boxes of A and B into a
//                      ring of shared-memory stages, completion on an mbarrier.
//   warp 1, one lane   MMA issuer: tcgen05.mma.kind::f8f6f4 (K = 32 per
//                      instruction) from shared-memory descriptors into one of
//                      two FP32 accumulators in tensor memory; tcgen05.commit
//                      releases the stage / publishes the tile.
//   warps 2..5         epilogue: tcgen05.ld of the finished accumulator (each
//                      warp owns the 32 TMEM lanes it may address), exact
//                      power-of-two unscale, optional bias vector, rounding,
//                      optional activation (second output) and amax, then
//                      swizzled shared-memory slabs and TMA stores (or direct
//                      stores for outputs whose rows are not 16-byte multiples).
// The epilogue comes in six kinds, a template parameter of both kernels so that
// each instantiation carries only its own arithmetic: plain; GELU forward; GELU
// backward; identity; SwiGLU forward; SwiGLU backward.  The five fused kinds
// write a second tensor z next to the (optional) matmul output -- as bf16
// and / or as FP8 bytes under a bias known before the launch -- and its amax;
// they run with one stage fewer and four staging slabs per epilogue warp.
// The two accumulators let the epilogue of tile i overlap the main loop of
// tile i+1.  An operand may be stored with the contraction index contiguous
// ("K-major": X8[T,K], W8[N,K] in the forward pass) or with its M / N index
// contiguous ("MN-major": the same buffers read by the backward matmuls); the
// difference is the shared-memory descriptor and the order of the TMA
// coordinates.  A and B may be different FP8 formats (E5 x E4 in the backward
// pass); formats and majorness live in the instruction descriptor.
//
// Every wait on an mbarrier is bounded: when it expires the CTA raises
// FP8_FLAG_TIMEOUT in the status word, all roles leave their loops, tensor
// memory is released and the kernel returns.
#include <cstdio>
#include <cstdlib>

#include "fp8lin_internal.cuh"
#include "ptx.cuh"
#include "cast_common.cuh"

namespace fp8lin {

constexpr int kBM = 128;          // rows of D per tile = TMEM lanes
constexpr int kBK = 128;          // contraction bytes per stage = one 128-byte swizzle row
constexpr int kUmmaK = 32;        // contraction elements per tcgen05.mma for 8-bit types
constexpr int kGemmThreads = 192;
constexpr int kGroupM = 16;       // tile rasterisation: m-blocks per group
constexpr int64_t kStreamOutBytes = 64ll << 20;   // outputs from this size on are stored with the evict-first mark
constexpr int kSlabBytes = 32 * 128;            // epilogue staging: 32 rows x 128 bytes, what one warp stores at a time
constexpr int kSingleSlabs = 2;                 // staging slabs per epilogue warp, single-CTA kernel
constexpr int kActSlabs = 4;                    // ... of the kernels with a second output: two {output, z} pairs
#ifndef FP8LIN_PAIR_SLABS
#define FP8LIN_PAIR_SLABS 2
#endif
constexpr int kPairSlabs = FP8LIN_PAIR_SLABS;   // ... and CTA-pair kernel

struct GemmParams {
    int M, N, K;
    int tiles_m, tiles_n, num_k;
    int group_m;                  // tile rasterisation: m-blocks per group
    int serpentine;               // pair kernel: every other tile of a pair walks the contraction backwards
    int out_stream;               // plain epilogue: the output is far larger than L2, its stores are marked evict-first
    int splits, kb_per_split;     // split-K (single-CTA kernel only): k-blocks per split
    float *partial;               // [splits, M, N] FP32 partial sums when splits > 1
    const int32_t *d_sa, *d_sb;   // paper-convention biases of the two operands
    int delta_sum;                // format shifts to add to them
    int a_mn, b_mn;               // operand stored with its M / N index contiguous (contraction index strided)
    int a_box_bytes;              // single-CTA kernel: bytes one A load brings (its box holds only the rows that exist)
    int dec_bn, dec_stages, dec_a_bytes;   // decode kernel: tile width, stages, bytes a stage sets aside for A
    int dec_cluster;              // decode kernel: CTAs of a cluster that share one tile's contraction (1: none)
    int early_b;                  // decode kernel: B may be read before the launch ahead of this one has completed
    int early_rings;              // ... how many rings of B tiles are requested then (the first into shared memory, the rest into L2)
    int col_lo;                   // direct stores skip columns below this one (0 except in the decode kernel's last tile)
    // decode kernel, activation quantised in the same launch (NULL / unused otherwise)
    const uint4 *qx;              // the bf16 activation [M, K], 16-byte vectors
    uint8_t *qx8;                 // out: its E4 bytes, which the A loads then read
    float *q_amax;                // out: its amax
    int32_t *q_bias;              // out: its scaling bias (paper convention)
    int q_margin, q_conv;
    int dbg;                      // experiments build only: timing variants that give wrong results
    const void *bias_vec;         // [N] or NULL
    int bias_dt;
    void *out;
    int out_dt;
    int64_t ldo;
    int vec_ok;                   // out 16-byte aligned and ldo*elem % 16 == 0
    int tma_out;                  // epilogue goes through shared memory and TMA stores (needs vec_ok)
    int act;                      // 0: plain epilogue.  Otherwise a second tensor z leaves with the output (out may be
                                  // NULL): 1: z = GELU of the bf16-rounded output; 2: z = the bf16-rounded output times
                                  // GELU'(aux); 3: z = the bf16-rounded output itself; 4: SwiGLU, the output's columns are
                                  // blocks of 32 gate columns followed by their 32 up columns and z[M, N/2] =
                                  // SiLU(gate) * up; 5: SwiGLU backward, the output is dz[M, N], aux[M, 2N] the stored
                                  // gate/up pre-activations in that block layout, z[M, 2N] their gradients likewise
    const void *aux;              // act == 2: [M, N] bf16, the pre-activation whose derivative scales the gradient
    int has_out2;                 // z is stored as bf16 through the second output map
    uint8_t *out8;                // or NULL: z also leaves as FP8 bytes [M, N], scaled by a bias known beforehand
    const int32_t *d_sq;          // ... that bias (paper convention, device memory)
    int q_fmt, delta_q;           // ... the format of the bytes and its shift
    unsigned *d_amax_bits;        // or NULL
    unsigned *d_status;
    uint32_t idesc;
    int no_loads;                 // measurement aid (fp8_selftest_mma_ceiling): the CTA-pair kernel issues no operand loads
};

// ---------------------------------------------------------------------------
// tcgen05 / TMEM wrappers (mbarrier and TMA wrappers live in ptx.cuh)
// ---------------------------------------------------------------------------

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_f8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                        uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor for a tile whose rows are 128 contiguous
// bytes along the contraction dimension, 128-byte swizzled, rows packed in
// groups of eight (1024 bytes apart): start address, leading offset 16 B
// (unused for swizzled layouts), stride offset 1024 B, descriptor version 1,
// layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// The same shared-memory rows read as an operand whose M / N index is the contiguous one ("MN-major"): a tile
// is [contraction rows][128 bytes of M or N], 128-byte swizzled; eight contraction rows form one 1024-byte
// group (stride offset), and a second block of 128 M / N values starts `lbo_bytes` further on (leading
// offset).  One tcgen05.mma (K = 32) consumes 32 rows = 4096 bytes.
__device__ __forceinline__ uint64_t smem_desc_mn128(uint32_t smem_addr, uint32_t lbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

__host__ __device__ inline uint32_t make_idesc(int a_fmt, int b_fmt, int n)
{
    // FP32 accumulate, both operands contraction-major, M = 128.
    return (1u << 4) | ((uint32_t)a_fmt << 7) | ((uint32_t)b_fmt << 10) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kBM >> 4) << 24);
}

// ---------------------------------------------------------------------------
// kernel
// ---------------------------------------------------------------------------

template <int BN, int STAGES, int SLABS = kSingleSlabs>
struct GemmSmem {
    static constexpr int kSlabs = SLABS;  // staging slabs per epilogue warp
    static constexpr int kABytes = kBM * kBK;
    static constexpr int kBBytes = BN * kBK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kEpiOffset = STAGES * kStageBytes;
    static constexpr int kBarOffset = kEpiOffset + 4 * SLABS * kSlabBytes;
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kTotal = kBarOffset + kNumBars * 8 + 16;
    static constexpr int kDynamic = kTotal + 1024;  // slack to align the base to 1024 B
    static constexpr int kTmemCols = (2 * BN < 32) ? 32 : 2 * BN;
};

__device__ __forceinline__ void tile_coords(int tile, const GemmParams &p, int &m_blk, int &n_blk)
{
    const int group = p.group_m * p.tiles_n;
    const int g = tile / group;
    const int first_m = g * p.group_m;
    const int gm = min(p.group_m, p.tiles_m - first_m);
    const int r = tile - g * group;
    m_blk = first_m + r % gm;
    n_blk = r / gm;
}

// Where in its k-range a tile of the single-CTA kernel starts (it wraps around): a different place per tile.
__device__ __forceinline__ int first_kblock(int m_blk, int n_blk, int len)
{
    return (int)(((unsigned)n_blk * 7u + (unsigned)m_blk * 3u) % (unsigned)len);
}

// One 32-column chunk of one accumulator row: unscale by the exact power of
// two, add the optional bias vector.
__device__ __forceinline__ void epilogue_values(const uint32_t (&r)[32], int col0, const GemmParams &p,
                                                const Pow2Pair sc, bool two_step, float (&v)[32])
{
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        v[i] = __uint_as_float(r[i]) * sc.first;
        if (two_step) v[i] *= sc.second;
    }
    if (p.bias_vec) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (col0 + i < p.N) {
                float b = p.bias_dt == FP8_F32
                              ? __ldg(reinterpret_cast<const float *>(p.bias_vec) + col0 + i)
                              : __uint_as_float(
                                    (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(p.bias_vec) + col0 + i) << 16);
                v[i] += b;
            }
        }
    }
}

// Round 32 values to bf16 pairs (memory order) and fold them into the running amax.
__device__ __forceinline__ void pack_bf16(const float (&v)[32], int col0, const GemmParams &p, uint32_t (&w)[16],
                                          uint32_t &amax_bits, bool row_ok)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(v[2 * i + 1]), "f"(v[2 * i]));
    if (p.d_amax_bits && row_ok) {
        if (col0 + 32 <= p.N) {  // whole chunk inside the tensor: both 16-bit lanes of a word at once
            uint32_t m2 = 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) m2 = __vmaxu2(m2, w[i] & 0x7FFF7FFFu);
            amax_bits = max(amax_bits, max(m2 & 0xFFFFu, m2 >> 16) << 16);
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                uint32_t a = w[i] & 0x7FFF7FFFu;
                if (col0 + 2 * i < p.N) amax_bits = max(amax_bits, (a & 0xFFFFu) << 16);
                if (col0 + 2 * i + 1 < p.N) amax_bits = max(amax_bits, a & 0xFFFF0000u);
            }
        }
    }
}
__device__ __forceinline__ void amax_f32(const float (&v)[32], int col0, const GemmParams &p, uint32_t &amax_bits,
                                         bool row_ok)
{
    if (p.d_amax_bits && row_ok) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < p.N) amax_bits = max(amax_bits, __float_as_uint(v[i]) & 0x7FFFFFFFu);
    }
}

// Direct stores from registers (any alignment, any N): one row per thread.
__device__ __forceinline__ void store_direct(const uint32_t (&r)[32], int row, int col0, const GemmParams &p,
                                             const Pow2Pair sc, bool two_step, uint32_t &amax_bits)
{
    if (row >= p.M || col0 >= p.N || col0 + 32 <= p.col_lo) return;
    float v[32];
    epilogue_values(r, col0, p, sc, two_step, v);
    const bool below = col0 < p.col_lo;   // the chunk starts in columns that another tile owns (decode kernel only)
    if (below) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < p.col_lo) v[i] = 0.0f;   // not stored; keeps them out of the amax
    }
    if (p.out_dt == FP8_BF16) {
        uint32_t w[16];
        pack_bf16(v, col0, p, w, amax_bits, true);
        uint16_t *dst = reinterpret_cast<uint16_t *>(p.out) + (int64_t)row * p.ldo + col0;
        if (p.vec_ok && col0 + 32 <= p.N && !below) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                reinterpret_cast<uint4 *>(dst)[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (col0 + i < p.N && col0 + i >= p.col_lo) dst[i] = (uint16_t)((i & 1) ? (w[i >> 1] >> 16) : (w[i >> 1] & 0xFFFFu));
        }
    } else {
        amax_f32(v, col0, p, amax_bits, true);
        float *dst = reinterpret_cast<float *>(p.out) + (int64_t)row * p.ldo + col0;
        if (p.vec_ok && col0 + 32 <= p.N && !below) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                reinterpret_cast<float4 *>(dst)[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (col0 + i < p.N && col0 + i >= p.col_lo) dst[i] = v[i];
        }
    }
}

// ---- staged epilogue: registers -> swizzled shared memory -> TMA store ----

__device__ __forceinline__ void tma_store_only(const CUtensorMap *map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(src), "r"(x), "r"(y)
                 : "memory");
}
// ... followed by its own commit: one bulk group per store
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(src), "r"(x), "r"(y)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The same store for an output far larger than L2: its lines are marked to leave L2 first, so that they do not push
// out operand strips that other CTAs are about to read.
__device__ __forceinline__ void tma_store_2d_stream(const CUtensorMap *map, uint32_t src, int x, int y)
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(src), "r"(x), "r"(y), "l"(pol)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// 16-byte piece j (0..7) of this lane's 128-byte row, at its 128-byte-swizzle position
__device__ __forceinline__ void slab_write(uint32_t slab, int lane, int j, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    const uint32_t addr = slab + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) << 4);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// Before a slab is overwritten, the store issued from it two slabs ago must have read it.
template <int NSLAB>
__device__ __forceinline__ void slab_acquire(int lane)
{
    // the store issued from this slab NSLAB slabs ago must have read it: at most NSLAB - 1 stores may be pending
    if (lane == 0) {
        if (NSLAB == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        else if (NSLAB == 3) asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory");
        else asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
    }
    __syncwarp();
}
__device__ __forceinline__ void slab_publish(const CUtensorMap *map, uint32_t slab, int lane, int x, int y, bool in_range,
                                             bool stream = false)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
        // One bulk group per slab use, store or no store: slab_acquire counts groups.  (A chunk beyond the last column
        // of a ragged tile used to commit nothing, so the count ran ahead and a slab could be rewritten while the
        // store of the tile's last real chunk was still reading it: seen as zeros in the last columns of a tensor,
        // in a few per cent of launches on a busy GPU.)
        if (!in_range) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        else if (stream) tma_store_2d_stream(map, slab, x, y);
        else tma_store_2d(map, slab, x, y);
    }
}

// Phi(-|x|), the lower tail of the standard normal distribution, and exp(-x^2 / 2), in about fifteen FP32
// instructions (the fused kernels run under the power cap: every epilogue instruction costs matmul time).
//   Phi(-|x|) = erfcx(z) / 2 * exp(-z^2),  z = |x| / sqrt 2,  erfcx(z) = exp(z^2) erfc(z),  erfcx(z) / 2 = t * Q(t),
//   t = 1 / (1 + z/2)
// Q is a degree-7 polynomial, a Chebyshev least-squares fit of erfcx(z) / (2t) over t in (0, 1] (all z >= 0) with
// relative error below 5e-6 -- relative, so that the far negative tail of GELU keeps its accuracy.  The
// exponential is the hardware's base-2 approximation, which flushes results below 2^-126 to zero; so it is
// taken 2^32 too large and Q's coefficients carry the 2^-32 (exactly), which keeps every product in range down
// to where GELU itself falls below the smallest bf16 subnormal (|x| > 14.2).
// Rounded to bf16, GELU(x) = max(x, 0) - |x| Phi(-|x|) differs from the correctly rounded value by at most one
// bf16 ulp (at 0.2 % of all bf16 inputs), and GELU'(x) stays within 1.2e-4 relative.
// (fit_normal_tail.py beside this file derives the coefficients and replays this arithmetic over every bf16 input.)
constexpr float kTwoM32 = 2.3283064365386963e-10f;  // 2^-32
__device__ __forceinline__ float rcp_approx(float v)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
// returns Phi(-|x|); gauss_2p32 = 2^32 * exp(-x^2 / 2)
__device__ __forceinline__ float normal_lower_tail(float x, float &gauss_2p32)
{
    const float t = rcp_approx(fmaf(fabsf(x), 0.35355339059327373f, 1.0f));
    float q = 0.0222922415f * kTwoM32;
    q = fmaf(q, t, -0.0444558002f * kTwoM32);
    q = fmaf(q, t, -0.0345738456f * kTwoM32);
    q = fmaf(q, t, 0.0718056038f * kTwoM32);
    q = fmaf(q, t, 0.078016676f * kTwoM32);
    q = fmaf(q, t, 0.124898158f * kTwoM32);
    q = fmaf(q, t, 0.140969709f * kTwoM32);
    q = fmaf(q, t, 0.141048044f * kTwoM32);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(gauss_2p32) : "f"(fmaf(x * x, -0.7213475204444817f, 32.0f)));
    return t * q * gauss_2p32;
}

// GELU(x) = x * Phi(x) = x/2 * (1 + erf(x / sqrt 2)) = max(x, 0) - |x| * Phi(-|x|)
__device__ __forceinline__ float gelu_f32(float x)
{
    float gauss;
    const float lower = normal_lower_tail(x, gauss);
    return fmaf(-fabsf(x), lower, fmaxf(x, 0.0f));
}

// 32 bf16 values (16 packed words): apply GELU to each, in FP32.
__device__ __forceinline__ void gelu_words(const uint32_t (&w)[16], float (&v)[32])
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        v[2 * i] = gelu_f32(__uint_as_float(w[i] << 16));
        v[2 * i + 1] = gelu_f32(__uint_as_float(w[i] & 0xFFFF0000u));
    }
}

// d/dx GELU(x) = Phi(x) + x * phi(x),  phi(x) = exp(-x^2 / 2) / sqrt(2 pi)
__device__ __forceinline__ float gelu_grad_f32(float x)
{
    float gauss_2p32;
    const float lower = normal_lower_tail(x, gauss_2p32);
    const float cdf = x > 0.0f ? 1.0f - lower : lower;
    return fmaf(x * (0.3989422804014327f * kTwoM32), gauss_2p32, cdf);
}

// 32 bf16 gradient values times GELU'(pre-activation), in FP32; `a` holds the 32 bf16 pre-activations.
__device__ __forceinline__ void gelu_backward_words(const uint32_t (&w)[16], const uint4 (&a)[4], float (&v)[32])
{
    const uint32_t *aw = reinterpret_cast<const uint32_t *>(a);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16) * gelu_grad_f32(__uint_as_float(aw[i] << 16));
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u) * gelu_grad_f32(__uint_as_float(aw[i] & 0xFFFF0000u));
    }
}

// sigma(a) = 1 / (1 + exp(-a)) with its relative accuracy kept in the negative tail: for a <= 0 it is e / (1 + e),
// e = exp(a), and e is taken 2^32 too large so that the hardware exponential (which flushes below 2^-126) stays in
// range down to where a * sigma(a) falls below the smallest bf16 subnormal.  Returns r = 1 / (1 + exp(-|a|)) and
// e_2p32 = 2^32 exp(-|a|); sigma(a) = r for a > 0, e_2p32 * r * 2^-32 otherwise.
__device__ __forceinline__ float sigmoid_parts(float a, float &e_2p32)
{
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e_2p32) : "f"(fmaf(fabsf(a), -1.4426950408889634f, 32.0f)));
    return rcp_approx(fmaf(e_2p32, kTwoM32, 1.0f));
}
// SiLU(a) = a * sigma(a)
__device__ __forceinline__ float silu_f32(float a)
{
    float e;
    const float r = sigmoid_parts(a, e);
    return a > 0.0f ? a * r : (a * e * r) * kTwoM32;
}
// SiLU(a) and d/da SiLU(a) = sigma + a sigma (1 - sigma)
__device__ __forceinline__ void silu_and_grad_f32(float a, float &silu, float &grad)
{
    float e;
    const float r = sigmoid_parts(a, e);
    const float sg = a > 0.0f ? r : (e * r) * kTwoM32;
    silu = a * sg;  // where sigma is subnormal (a < -87) the product is below every bf16 normal anyway
    grad = fmaf(silu, 1.0f - sg, sg);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Four bf16 values (two packed words, memory order) scaled by the exact power of two and rounded to four FP8 bytes,
// as cast4 does; instead of testing each value for clipping, the largest scaled magnitude is kept in `peak` and
// tested once per tile (the epilogue pays for every instruction per element).
template <int FMT, bool TWO_STEP>
__device__ __forceinline__ uint32_t quantise4(uint32_t w0, uint32_t w1, const Pow2Pair p, float &peak)
{
    float f0 = bf16_lo(w0) * p.first, f1 = bf16_hi(w0) * p.first, f2 = bf16_lo(w1) * p.first, f3 = bf16_hi(w1) * p.first;
    if (TWO_STEP) {
        f0 *= p.second; f1 *= p.second; f2 *= p.second; f3 *= p.second;
    }
    peak = fmaxf(fmaxf(peak, fabsf(f0)), fmaxf(fmaxf(fabsf(f1), fabsf(f2)), fabsf(f3)));
    return cvt_pair<FMT>(f1, f0) | (cvt_pair<FMT>(f3, f2) << 16);
}
// n words of bf16 pairs -> n/2 words of FP8 bytes
template <int FMT, int NW>
__device__ __forceinline__ void quantise_words(const uint32_t (&w)[NW], uint32_t *b8, const Pow2Pair p, bool two_step,
                                               float &peak)
{
    if (two_step) {
#pragma unroll
        for (int i = 0; i < NW / 2; ++i) b8[i] = quantise4<FMT, true>(w[2 * i], w[2 * i + 1], p, peak);
    } else {
#pragma unroll
        for (int i = 0; i < NW / 2; ++i) b8[i] = quantise4<FMT, false>(w[2 * i], w[2 * i + 1], p, peak);
    }
}
// the saturation rule of the cast kernels on the largest scaled magnitude
template <int FMT>
__device__ __forceinline__ bool peak_clips(float peak)
{
    return FMT == FP8_E4 ? peak > 464.0f : peak >= 61440.0f;
}

// One warp's share (32 rows x BN columns) of a finished accumulator.
//   t_row        TMEM address of this warp's lanes at the accumulator's first column
//   row0         first of the warp's 32 output rows;  col_base  first output column of the tile
//   release_bar  barrier to arrive on once the accumulator has been read (cluster address if remote)
template <int BN, int ACT, int NSLAB>
__device__ __forceinline__ void epilogue_tile(const CUtensorMap *map_out, const CUtensorMap *map_out2, uint32_t t_row,
                                              int row0, int col_base,
                                              const GemmParams &p, const Pow2Pair sc, bool two_step,
                                              uint32_t &amax_bits, uint32_t warp_slabs, uint32_t &slab_count,
                                              uint32_t release_bar, bool release_remote, int lane)
{
    auto release = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (release_remote)
                asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(release_bar) : "memory");
            else
                mbar_arrive(release_bar);
        }
    };
    if (!p.tma_out) {
        if (row0 >= p.M) {   // none of this warp's rows exists (decode): nothing to read
            release();
            return;
        }
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            uint32_t r[32];
            tmem_ld_x32(t_row + c, r);
            tmem_ld_wait();
            if (c + 32 >= BN) release();
            store_direct(r, row0 + lane, col_base + c, p, sc, two_step, amax_bits);
        }
        return;
    }
    const bool rows_in = row0 < p.M;
    const bool row_ok = row0 + lane < p.M;
    if constexpr (ACT == 4) {
        // SwiGLU forward.  Chunks of 32 accumulator columns alternate gate, up, gate, up ...; the gate chunk's bf16
        // words wait in registers for their up chunk; 32 z values come out of every pair of chunks, so one slab row
        // of z (64 columns) covers 128 accumulator columns.  Slabs 0 and 2 stage the pre-activation (alternating
        // per 64 columns), slabs 1 and 3 stage z (alternating per 128 columns); one bulk group per 64 columns.
        static_assert(NSLAB == 4, "SwiGLU epilogue needs four slabs per warp");
        uint32_t dummy = 0, wg[16];
        float peak = 0.0f;
        Pow2Pair scq = make_pow2_pair(0);
        bool scq_two = false;
        if (p.out8) {
            const int sq = __ldcg(p.d_sq) + p.delta_q;
            scq = make_pow2_pair(sq);
            scq_two = sq < -126 || sq > 127;
        }
        const int64_t ldz = p.ldo >> 1;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            const int h = (c >> 5) & 1, pc = c >> 6;
            uint32_t r[32];
            tmem_ld_x32(t_row + c, r);
            tmem_ld_wait();
            if (c + 32 >= BN) release();
            const uint32_t slab_pre = warp_slabs + (pc & 1) * 2 * kSlabBytes;
            const uint32_t slab_z = warp_slabs + (((pc >> 1) & 1) * 2 + 1) * kSlabBytes;
            if (h == 0) {
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                __syncwarp();
            }
            const int col0 = col_base + c;
            float v[32];
            uint32_t w[16];
            epilogue_values(r, col0, p, sc, two_step, v);
            pack_bf16(v, col0, p, w, dummy, false);
            if (p.out) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    slab_write(slab_pre, lane, 4 * h + j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            }
            if (h == 0) {
#pragma unroll
                for (int i = 0; i < 16; ++i) wg[i] = w[i];
                continue;
            }
            // up chunk: z = SiLU(gate) * up on the bf16-rounded pre-activations
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                v[2 * i] = silu_f32(bf16_lo(wg[i])) * bf16_lo(w[i]);
                v[2 * i + 1] = silu_f32(bf16_hi(wg[i])) * bf16_hi(w[i]);
            }
            const bool in_n = col0 < p.N;  // N is a multiple of 64: a gate/up pair of chunks is whole or absent
            uint32_t wz[16];
            pack_bf16(v, col0, p, wz, amax_bits, row_ok && in_n);
            const int zc = (col0 - 32) >> 1;  // first of the 32 z columns
            if (p.has_out2) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    slab_write(slab_z, lane, 4 * (pc & 1) + j, wz[4 * j], wz[4 * j + 1], wz[4 * j + 2], wz[4 * j + 3]);
            }
            if (p.out8 && row_ok && in_n) {
                uint32_t b8[8];
                quantise_words<FP8_E4>(wz, b8, scq, scq_two, peak);
                uint8_t *dst = p.out8 + (int64_t)(row0 + lane) * ldz + zc;
                reinterpret_cast<uint4 *>(dst)[0] = make_uint4(b8[0], b8[1], b8[2], b8[3]);
                reinterpret_cast<uint4 *>(dst)[1] = make_uint4(b8[4], b8[5], b8[6], b8[7]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (rows_in && in_n && p.out) tma_store_only(map_out, slab_pre, col0 - 32, row0);
                // the z slab leaves after its second half, or after its first when the tensor ends there
                const bool last_half = (pc & 1) || col0 + 32 >= p.N;
                const int z0 = (col_base + (pc & ~1) * 64) >> 1;
                if (rows_in && p.has_out2 && last_half && z0 < (p.N >> 1)) tma_store_only(map_out2, slab_z, z0, row0);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        }
        if (__any_sync(0xFFFFFFFFu, peak_clips<FP8_E4>(peak)) && lane == 0) atomicOr(p.d_status, (unsigned)FP8_FLAG_SATURATED);
        return;
    }
    if constexpr (ACT == 5) {
        // SwiGLU backward.  Every 32 accumulator columns (dz) give 64 output columns: the gradients of their 32
        // gate and 32 up pre-activations, one full slab row.  Slabs 0 and 2 stage dz (alternating per 64 columns),
        // slabs 1 and 3 the gradients (alternating per 32 columns); one bulk group per 32 columns.
        static_assert(NSLAB == 4, "SwiGLU epilogue needs four slabs per warp");
        uint32_t dummy = 0;
        float peak = 0.0f;
        Pow2Pair scq = make_pow2_pair(0);
        bool scq_two = false;
        if (p.out8) {
            const int sq = __ldcg(p.d_sq) + p.delta_q;
            scq = make_pow2_pair(sq);
            scq_two = sq < -126 || sq > 127;
        }
        const int64_t ld2 = p.ldo * 2;
        // the stored pre-activations of a chunk (32 gate values then 32 up values, 128 bytes per row) are requested
        // one chunk ahead, so that their trip from memory overlaps the arithmetic of the chunk before
        uint4 aux_next[8];
        auto fetch_aux = [&](int c) {
            const int col0 = col_base + c;
            const bool ok = row_ok && col0 < p.N;
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(p.aux) +
                                                               (int64_t)(row0 + lane) * ld2 + 2 * (int64_t)col0);
#pragma unroll
            for (int j = 0; j < 8; ++j) aux_next[j] = ok ? __ldg(src + j) : make_uint4(0, 0, 0, 0);
        };
        fetch_aux(0);
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            const int h = (c >> 5) & 1, pc = c >> 6;
            uint32_t r[32];
            tmem_ld_x32(t_row + c, r);
            uint4 aux_now[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) aux_now[j] = aux_next[j];
            if (c + 32 < BN) fetch_aux(c + 32);
            tmem_ld_wait();
            if (c + 32 >= BN) release();
            const uint32_t slab_dz = warp_slabs + (pc & 1) * 2 * kSlabBytes;
            const uint32_t slab_g = warp_slabs + (h * 2 + 1) * kSlabBytes;
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            __syncwarp();
            const int col0 = col_base + c;
            const bool in_n = col0 < p.N;  // N is a multiple of 32: a chunk is whole or absent
            float v[32];
            uint32_t w[16];
            epilogue_values(r, col0, p, sc, two_step, v);
            pack_bf16(v, col0, p, w, dummy, false);
            if (p.out) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    slab_write(slab_dz, lane, 4 * h + j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            }
            // the stored pre-activations of these 32 features: 32 gate values then 32 up values, 128 bytes
            const bool ok = row_ok && in_n;
            uint32_t wgr[16], wur[16];
            {
                const uint32_t *ag = reinterpret_cast<const uint32_t *>(aux_now);  // 16 words of gate, 16 of up
                float vg[32];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float s0, d0, s1, d1;
                    silu_and_grad_f32(bf16_lo(ag[i]), s0, d0);
                    silu_and_grad_f32(bf16_hi(ag[i]), s1, d1);
                    const float z0 = bf16_lo(w[i]), z1 = bf16_hi(w[i]);
                    vg[2 * i] = z0 * bf16_lo(ag[16 + i]) * d0;
                    vg[2 * i + 1] = z1 * bf16_hi(ag[16 + i]) * d1;
                    v[2 * i] = z0 * s0;
                    v[2 * i + 1] = z1 * s1;
                }
                pack_bf16(vg, col0, p, wgr, amax_bits, ok);
                pack_bf16(v, col0, p, wur, amax_bits, ok);
            }
            if (p.has_out2) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    slab_write(slab_g, lane, j, wgr[4 * j], wgr[4 * j + 1], wgr[4 * j + 2], wgr[4 * j + 3]);
                    slab_write(slab_g, lane, 4 + j, wur[4 * j], wur[4 * j + 1], wur[4 * j + 2], wur[4 * j + 3]);
                }
            }
            if (p.out8 && ok) {
                uint32_t b8[16];
                quantise_words<FP8_E5>(wgr, b8, scq, scq_two, peak);
                quantise_words<FP8_E5>(wur, b8 + 8, scq, scq_two, peak);
                uint4 *dst = reinterpret_cast<uint4 *>(p.out8 + (int64_t)(row0 + lane) * ld2 + 2 * (int64_t)col0);
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[j] = make_uint4(b8[4 * j], b8[4 * j + 1], b8[4 * j + 2], b8[4 * j + 3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (rows_in && in_n) {
                    if (p.has_out2) tma_store_only(map_out2, slab_g, 2 * col0, row0);
                    if (p.out && (h == 1 || col0 + 32 >= p.N)) tma_store_only(map_out, slab_dz, col0 - 32 * h, row0);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        }
        if (__any_sync(0xFFFFFFFFu, peak_clips<FP8_E5>(peak)) && lane == 0) atomicOr(p.d_status, (unsigned)FP8_FLAG_SATURATED);
        return;
    }
    if (ACT) {
        // The pre-activation (optional) and the second tensor z leave together, 64 columns (one 128-byte slab row
        // each) at a time; the warp's slabs are used in pairs {pre, z} in rotation.  The loop body covers 32
        // columns and is not unrolled: fully unrolled, the activation arithmetic outgrows the instruction cache.
        constexpr int kPairsOfSlabs = NSLAB / 2;
        uint32_t dummy = 0;
        float peak = 0.0f;
        Pow2Pair scq = make_pow2_pair(0);
        bool scq_two = false;
        if (p.out8) {
            const int sq = __ldcg(p.d_sq) + p.delta_q;
            scq = make_pow2_pair(sq);
            scq_two = sq < -126 || sq > 127;
        }
        // ACT == 2: the stored pre-activations of a chunk (64 bytes per row) are requested one chunk ahead, so that
        // their trip from memory overlaps the arithmetic of the chunk before
        uint4 aux_next[4];
        auto fetch_aux = [&](int c) {
            const int col0 = col_base + c;
            const bool ok = row_ok && col0 + 32 <= p.N;
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(p.aux) +
                                                               (int64_t)(row0 + lane) * p.ldo + col0);
#pragma unroll
            for (int j = 0; j < 4; ++j) aux_next[j] = ok ? __ldg(src + j) : make_uint4(0, 0, 0, 0);
        };
        if (ACT == 2) fetch_aux(0);
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            const int h = (c >> 5) & 1;  // which half of the slab rows
            uint32_t r[32];
            tmem_ld_x32(t_row + c, r);
            uint4 aux_now[4];
            if (ACT == 2) {
#pragma unroll
                for (int j = 0; j < 4; ++j) aux_now[j] = aux_next[j];
                if (c + 32 < BN) fetch_aux(c + 32);
            }
            tmem_ld_wait();
            if (c + 32 >= BN) release();
            const uint32_t slab_pre = warp_slabs + (slab_count % kPairsOfSlabs) * 2 * kSlabBytes;
            const uint32_t slab_act = slab_pre + kSlabBytes;
            if (h == 0) {
                // one bulk group per 64 columns: the group that last read this pair of slabs must have finished
                if (lane == 0) {
                    if (kPairsOfSlabs == 1) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    else asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                }
                __syncwarp();
            }
            const int col0 = col_base + c;
            float v[32];
            uint32_t w[16], wa[16];
            epilogue_values(r, col0, p, sc, two_step, v);
            pack_bf16(v, col0, p, w, dummy, false);
            if (p.out) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    slab_write(slab_pre, lane, 4 * h + j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            }
            if (ACT == 1) {
                gelu_words(w, v);  // the activation sees exactly what the pre-activation tensor holds
            } else if (ACT == 3) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    v[2 * i] = __uint_as_float(w[i] << 16);
                    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
                }
            } else {
                // columns beyond N are clipped by the store; rows beyond M have no pre-activation to read
                const bool ok = row_ok && col0 + 32 <= p.N;
                gelu_backward_words(w, aux_now, v);
                if (row_ok && !ok && col0 < p.N) {   // ragged last chunk: element by element
                    const uint16_t *ar = reinterpret_cast<const uint16_t *>(p.aux) + (int64_t)(row0 + lane) * p.ldo;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float g = (i & 1) ? __uint_as_float(w[i >> 1] & 0xFFFF0000u) : __uint_as_float(w[i >> 1] << 16);
                        v[i] = col0 + i < p.N ? g * gelu_grad_f32(__uint_as_float((uint32_t)__ldg(ar + col0 + i) << 16)) : 0.0f;
                    }
                }
            }
            pack_bf16(v, col0, p, wa, amax_bits, row_ok);
            if (p.has_out2) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    slab_write(slab_act, lane, 4 * h + j, wa[4 * j], wa[4 * j + 1], wa[4 * j + 2], wa[4 * j + 3]);
            }
            if (p.out8 && row_ok && col0 < p.N) {
                // the bytes are made from the bf16 values just rounded, as a cast of the stored tensor would;
                // one row per lane, 32 bytes
                uint32_t b8[8];
                if (p.q_fmt == FP8_E4) quantise_words<FP8_E4>(wa, b8, scq, scq_two, peak);
                else quantise_words<FP8_E5>(wa, b8, scq, scq_two, peak);
                uint8_t *dst = p.out8 + (int64_t)(row0 + lane) * p.ldo + col0;
                if (col0 + 32 <= p.N) {
                    reinterpret_cast<uint4 *>(dst)[0] = make_uint4(b8[0], b8[1], b8[2], b8[3]);
                    reinterpret_cast<uint4 *>(dst)[1] = make_uint4(b8[4], b8[5], b8[6], b8[7]);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (col0 + i < p.N) dst[i] = (uint8_t)(b8[i >> 2] >> (8 * (i & 3)));
                }
            }
            if (h == 1) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    const int x = col0 - 32;
                    if (rows_in && x < p.N) {
                        if (p.out) tma_store_only(map_out, slab_pre, x, row0);
                        if (p.has_out2) tma_store_only(map_out2, slab_act, x, row0);
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                ++slab_count;
            }
        }
        const bool clipped = p.q_fmt == FP8_E4 ? peak_clips<FP8_E4>(peak) : peak_clips<FP8_E5>(peak);
        if (__any_sync(0xFFFFFFFFu, clipped) && lane == 0) atomicOr(p.d_status, (unsigned)FP8_FLAG_SATURATED);
        return;
    }
    if (p.out_dt == FP8_BF16) {
#pragma unroll 1
        for (int c = 0; c < BN; c += 64) {  // one slab = 64 bf16 columns
            uint32_t r0[32], r1[32];
            tmem_ld_x32(t_row + c, r0);
            tmem_ld_x32(t_row + c + 32, r1);
            tmem_ld_wait();
#ifdef FP8LIN_EXPERIMENTS
            // timing only (wrong results): the accumulator is handed back after its first 64 columns have been read,
            // which bounds what an earlier release could be worth
            if (p.dbg == 21 ? c == 0 : c + 64 >= BN) release();
#else
            if (c + 64 >= BN) release();
#endif

            const uint32_t slab = warp_slabs + (slab_count % NSLAB) * kSlabBytes;
            ++slab_count;
            slab_acquire<NSLAB>(lane);
            float v[32];
            uint32_t w[16];
            epilogue_values(r0, col_base + c, p, sc, two_step, v);
            pack_bf16(v, col_base + c, p, w, amax_bits, row_ok);
#pragma unroll
            for (int j = 0; j < 4; ++j) slab_write(slab, lane, j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            epilogue_values(r1, col_base + c + 32, p, sc, two_step, v);
            pack_bf16(v, col_base + c + 32, p, w, amax_bits, row_ok);
#pragma unroll
            for (int j = 0; j < 4; ++j) slab_write(slab, lane, 4 + j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            slab_publish(map_out, slab, lane, col_base + c, row0, rows_in && col_base + c < p.N, p.out_stream != 0);
        }
    } else {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {  // one slab = 32 fp32 columns
            uint32_t r[32];
            tmem_ld_x32(t_row + c, r);
            tmem_ld_wait();
            if (c + 32 >= BN) release();
            const uint32_t slab = warp_slabs + (slab_count % NSLAB) * kSlabBytes;
            ++slab_count;
            slab_acquire<NSLAB>(lane);
            float v[32];
            epilogue_values(r, col_base + c, p, sc, two_step, v);
            amax_f32(v, col_base + c, p, amax_bits, row_ok);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                slab_write(slab, lane, j, __float_as_uint(v[4 * j]), __float_as_uint(v[4 * j + 1]),
                           __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
            slab_publish(map_out, slab, lane, col_base + c, row0, rows_in && col_base + c < p.N, p.out_stream != 0);
        }
    }
}

// The i-th work item of a CTA of the single-CTA kernel: an output tile and a slice [k0, k1) of its contraction.
// Ordinary launches deal (tile, slice) pairs round-robin to the CTAs.  The FP16-accumulation kind (ACT == 6) keeps
// all slices of a tile on one CTA, in order: its epilogue folds them into a running FP16 sum one after the other.
template <int ACT>
__device__ __forceinline__ bool item_at(const GemmParams &p, int i, int &tile, int &split)
{
    if (ACT == 6) {
        tile = (int)blockIdx.x + (i / p.splits) * (int)gridDim.x;
        split = i % p.splits;
        return tile < p.tiles_m * p.tiles_n;
    }
    const int item = (int)blockIdx.x + i * (int)gridDim.x;
    tile = item / p.splits;
    split = item % p.splits;
    return item < p.tiles_m * p.tiles_n * p.splits;
}

// FP16 accumulation (Fig. 3b, Section 2.4): the accumulator of one slice (the exact-to-FP32 sum of `chunk` products
// per output) is added to a running FP16 sum with one rounding to FP16 per slice; after the last slice the FP16 sum
// is unscaled in FP16 (Eq. 2 on an FP16 output) and stored.  The running sums of the CTA's 128 x 256 tile live in
// shared memory as [32-column chunk][16-byte piece][row]: a warp's 32 rows are 512 contiguous bytes, no conflicts.
template <int BN>
__device__ __forceinline__ void epilogue_f16acc(uint32_t t_row, int row, int col_base, const GemmParams &p, const Pow2Pair sc,
                                                uint32_t acc_smem, int local_row, bool first, bool last,
                                                uint32_t release_bar, int lane)
{
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
        uint32_t r[32];
        tmem_ld_x32(t_row + c, r);
        tmem_ld_wait();
        if (c + 32 >= BN) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(release_bar);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t addr = acc_smem + (uint32_t)((((c >> 5) * 4 + j) * kBM + local_row) * 16);
            uint32_t h[4] = {0u, 0u, 0u, 0u};
            if (!first) asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]) : "r"(addr));
            float out[8];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                float lo, hi;
                asm("{ .reg .b16 l, u; mov.b32 {l, u}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, u; }" : "=f"(lo), "=f"(hi) : "r"(h[w]));
                lo += __uint_as_float(r[8 * j + 2 * w]);       // running FP16 sum + this slice's partial sum ...
                hi += __uint_as_float(r[8 * j + 2 * w + 1]);
                asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h[w]) : "f"(hi), "f"(lo));   // ... rounded to FP16, once per slice
                if (last) {
                    asm("{ .reg .b16 l, u; mov.b32 {l, u}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, u; }" : "=f"(lo), "=f"(hi) : "r"(h[w]));
                    out[2 * w] = lo * sc.first * sc.second;    // exact power of two; the FP16 rounding below is the only one
                    out[2 * w + 1] = hi * sc.first * sc.second;
                }
            }
            if (!last) {
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(h[0]), "r"(h[1]), "r"(h[2]), "r"(h[3]) : "memory");
                continue;
            }
            const int col0 = col_base + c + 8 * j;
            if (row >= p.M || col0 >= p.N) continue;   // N is a multiple of 8: a piece is whole or absent
            uint32_t o16[4];
#pragma unroll
            for (int w = 0; w < 4; ++w) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(o16[w]) : "f"(out[2 * w + 1]), "f"(out[2 * w]));
            if (p.out_dt == FP8_F16) {
                *reinterpret_cast<uint4 *>(reinterpret_cast<uint16_t *>(p.out) + (int64_t)row * p.ldo + col0) =
                    make_uint4(o16[0], o16[1], o16[2], o16[3]);
            } else {   // FP32 holding exactly the FP16 values
                float f[8];
#pragma unroll
                for (int w = 0; w < 4; ++w)
                    asm("{ .reg .b16 l, u; mov.b32 {l, u}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, u; }" : "=f"(f[2 * w]), "=f"(f[2 * w + 1]) : "r"(o16[w]));
                float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out) + (int64_t)row * p.ldo + col0);
                dst[0] = make_float4(f[0], f[1], f[2], f[3]);
                dst[1] = make_float4(f[4], f[5], f[6], f[7]);
            }
        }
    }
}

template <int BN, int STAGES, int ACT>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_out2,
            const GemmParams p)
{
    using L = GemmSmem<BN, STAGES, ACT ? kActSlabs : kSingleSlabs>;   // ACT == 6: the 64 KB of the four slabs per warp hold the FP16 sums
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOffset + L::kNumBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), L::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The finalize kernel of a split contraction is launched as a programmatic dependent: its CTAs may take
    // their places now and wait, at their first instruction, for this grid to complete and flush.
    if (p.splits > 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
            uint32_t it = 0;
            bool alive = true;
            // One row of tiles (decode): every B byte is read exactly once, every A byte by every CTA.  B is marked
            // to leave L2 first and A to stay: without the hints the few lines of A can lose their place to the
            // streaming weights and every CTA then fetches them from one DRAM page (measured: 88 -> 140 us for a
            // 470 MB weight, depending on where the activation happened to be allocated).
            const bool stream_b = p.tiles_m == 1;
            const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
            auto load_b = [&](int s, int n_blk, int k) {
                const uint32_t b_dst = smem_base + s * L::kStageBytes + L::kABytes;
                if (p.b_mn) {  // two blocks of 128 N values, 16 KB apart
                    for (int h = 0; h < BN / 128; ++h) {
                        if (stream_b)
                            tma_load_2d_hint(b_dst + h * (128 * kBK), &map_b, full_bar(s), n_blk * BN + h * 128, k * kBK, drop);
                        else
                            tma_load_2d(b_dst + h * (128 * kBK), &map_b, full_bar(s), n_blk * BN + h * 128, k * kBK);
                    }
                } else if (stream_b) {
                    tma_load_2d_hint(b_dst, &map_b, full_bar(s), k * kBK, n_blk * BN, drop);
                } else {
                    tma_load_2d(b_dst, &map_b, full_bar(s), k * kBK, n_blk * BN);
                }
            };
            // When this grid runs as a programmatic dependent of the launch before it (a decode-size cast), nothing
            // that launch may have written is read before it has completed; but the first ring of B tiles (the
            // weights, in decode) is already pulled towards L2, which holds no stale data whoever writes them.
            int tile0, split0;
            if (item_at<ACT>(p, 0, tile0, split0)) {
                int m_blk, n_blk;
                tile_coords(tile0, p, m_blk, n_blk);
                const int k0 = split0 * p.kb_per_split;
                const int k1 = min(p.num_k, k0 + p.kb_per_split);
                int k = k0 + first_kblock(m_blk, n_blk, k1 - k0);
                for (int i = 0; i < min(k1 - k0, STAGES); ++i, k = (k + 1 == k1) ? k0 : k + 1) {
                    if (p.b_mn) {
                        for (int h = 0; h < BN / 128; ++h) tma_prefetch_l2_2d(&map_b, n_blk * BN + h * 128, k * kBK);
                    } else {
                        tma_prefetch_l2_2d(&map_b, k * kBK, n_blk * BN);
                    }
                }
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int tile, split;
            for (int i = 0; alive && item_at<ACT>(p, i, tile, split); ++i) {
                int m_blk, n_blk;
                tile_coords(tile, p, m_blk, n_blk);
                const int k0 = split * p.kb_per_split;
                const int k1 = min(p.num_k, k0 + p.kb_per_split);
                // The k-blocks of an item are taken in a rotated order that differs from tile to tile: with a few
                // rows of A, all CTAs walking k in step would ask L2 for the same 128-byte lines at the same time
                // (measured on 1 to 8 rows: 103-109 us against 83-86 us for a 470 MB weight).
                int k = k0 + first_kblock(m_blk, n_blk, k1 - k0);
                for (int i = 0; i < k1 - k0; ++i, ++it, k = (k + 1 == k1) ? k0 : k + 1) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.d_status)) { alive = false; break; }
                    mbar_expect_tx(full_bar(s), (uint32_t)p.a_box_bytes + L::kBBytes);
                    const uint32_t a_dst = smem_base + s * L::kStageBytes;
                    if (stream_b) {
                        if (p.a_mn) tma_load_2d_hint(a_dst, &map_a, full_bar(s), m_blk * kBM, k * kBK, keep);
                        else tma_load_2d_hint(a_dst, &map_a, full_bar(s), k * kBK, m_blk * kBM, keep);
                    } else {
                        if (p.a_mn) tma_load_2d(a_dst, &map_a, full_bar(s), m_blk * kBM, k * kBK);
                        else tma_load_2d(a_dst, &map_a, full_bar(s), k * kBK, m_blk * kBM);
                    }
                    load_b(s, n_blk, k);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, t = 0;
            bool alive = true;
            // the bounded waits below start counting only once the launch before this one has completed
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int tile, split;
            for (int i = 0; alive && item_at<ACT>(p, i, tile, split); ++i, ++t) {
                const int k0 = split * p.kb_per_split;
                const int k1 = min(p.num_k, k0 + p.kb_per_split);
                const int buf = t & 1;
                const uint32_t acc_ph = (t >> 1) & 1u;
                if (!mbar_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, p.d_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int k = k0; k < k1; ++k, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.d_status)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * L::kStageBytes;
                    const uint64_t da = p.a_mn ? smem_desc_mn128(a_addr, 128 * kBK) : smem_desc_k128(a_addr);
                    const uint64_t db = p.b_mn ? smem_desc_mn128(a_addr + L::kABytes, 128 * kBK)
                                               : smem_desc_k128(a_addr + L::kABytes);
                    // per instruction (K = 32): 32 bytes along a 128-byte row, or 32 rows = 4096 bytes
                    const uint32_t step_a = p.a_mn ? 256u : 2u, step_b = p.b_mn ? 256u : 2u;
#pragma unroll
                    for (int j = 0; j < kBK / kUmmaK; ++j)
                        umma_f8(d_tmem, da + step_a * j, db + step_b * j, p.idesc, (k > k0 || j > 0) ? 1u : 0u);
                    umma_commit(empty_bar(s));
                }
                if (alive) umma_commit(acc_full_bar(buf));
            }
        }
    } else {
        // ------------------------------- epilogue -------------------------------
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the biases may come from the launch before this one
        const int q = warp & 3;  // TMEM lane quarter this warp may address
        const int e = -(__ldcg(p.d_sa) + __ldcg(p.d_sb) + p.delta_sum);
        const Pow2Pair sc = make_pow2_pair(e);
        const bool two_step = (e < -126 || e > 127);
        uint32_t amax_bits = 0, slab_count = 0;
        const uint32_t warp_slabs = smem_base + L::kEpiOffset + q * L::kSlabs * kSlabBytes;
        uint32_t t = 0;
        // with split-K every item leaves its raw FP32 partial sum in the workspace; a second kernel finishes
        GemmParams pp = p;
        if (ACT != 6 && p.splits > 1) {
            pp.out_dt = FP8_F32;
            pp.out_stream = 0;   // the partial sums are read back at once
            pp.bias_vec = nullptr;
            pp.d_amax_bits = nullptr;
            pp.tma_out = 0;
            pp.vec_ok = (p.N % 4) == 0;
        }
        const Pow2Pair sc_one = make_pow2_pair(0);
        int tile, split;
        for (int i = 0; item_at<ACT>(p, i, tile, split); ++i, ++t) {
            int m_blk, n_blk;
            tile_coords(tile, p, m_blk, n_blk);
            if (ACT != 6 && p.splits > 1) pp.out = p.partial + (int64_t)split * p.M * p.N;
            const int buf = t & 1;
            const uint32_t acc_ph = (t >> 1) & 1u;
            // every lane waits (each needs the ordering), but the warp leaves together
            const bool ready = mbar_wait(acc_full_bar(buf), acc_ph, abort_flag, p.d_status);
            if (!__all_sync(0xFFFFFFFFu, ready)) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN;
            if constexpr (ACT == 6) {
                epilogue_f16acc<BN>(t_row, m_blk * kBM + q * 32 + lane, n_blk * BN, p, sc, smem_base + L::kEpiOffset, q * 32 + lane,
                                    split == 0, split == p.splits - 1, acc_empty_bar(buf), lane);
                continue;
            }
            epilogue_tile<BN, ACT, L::kSlabs>(&map_out, &map_out2, t_row, m_blk * kBM + q * 32, n_blk * BN, pp,
                              p.splits > 1 ? sc_one : sc, p.splits > 1 ? false : two_step, amax_bits, warp_slabs, slab_count,
                              acc_empty_bar(buf), false, lane);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        if (p.d_amax_bits) {
            amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
            if (lane == 0 && amax_bits) atomicMax(p.d_amax_bits, amax_bits);
        }
    }

    // ------------------------------- teardown -------------------------------
    __syncwarp();  // the single-lane roles rejoin their warps before the block-wide barrier
    if (*abort_flag) __nanosleep(20000);  // let copies and MMAs already issued drain before the memory is released
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, L::kTmemCols);
}


// ---------------------------------------------------------------------------
// Decode kernel: at most 128 rows of A, both operands contraction-major, plain epilogue
// ---------------------------------------------------------------------------
//
// The weight-streaming regime (Section 3.1: weights quantised once, a few activation rows per call).  Same pipeline
// as gemm_kernel, with the tile width and the stage count chosen per launch instead of per instantiation: the host
// picks a width `bn` (a multiple of 16 up to 256) that gives close to one tile per SM, so that most layers need no
// split contraction (no partial sums, no second launch), and as many stages as shared memory holds, so that a CTA
// keeps about 190 KB of weight bytes in flight whatever the width.  A stage is `a_bytes` of A (the rows that exist,
// rounded up to the 1024-byte swizzle atom; the instruction reads 128 rows, the rest being the head of the B tile
// behind it, feeding output rows that are never stored) followed by bn x 128 bytes of B.  The few output rows are
// stored from registers.
//
// Where a layer has too few tiles for the SMs, the contraction of a tile is split across the CTAs of a cluster
// (p.dec_cluster of them, one item each): when all have finished their slices the others write their FP32 sums
// into the leader's shared memory (its stages are free by then) and the leader adds them in rank order and stores
// the result: no partial sums in global memory, no second launch.  Two cluster barriers frame the exchange; a CTA
// whose wait ran out still takes part in both.
//
// With p.qx set the launch also quantises the activation (FP8-AMAX, Eq. 3 and Eq. 1, bit for bit what fp8_cast_e4
// does), for activations of a few rows (at most 64 KB): after the dependency wait the four epilogue warps of EVERY CTA
// take the amax of the whole of X, derive the bias, cast the whole of X and write the bytes (every CTA writes the same
// bytes to the same places; each reads back only what it has itself written), and only then does the producer start
// the A loads (its weight tiles have been streaming since the kernel began).  No CTA waits for another: the small
// cast kernel, its launch and two dependency hops leave the critical path at the price of reading 64 KB from L2 per
// CTA.  (A version that shared the work between the CTAs, with two barriers across the grid, was slower than the
// separate cast kernel: 177 against 165 us for a four-layer decoder block at one row.)

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

#ifdef FP8LIN_EXPERIMENTS
// timeline of the decode launches (block 0): entry, dependency wait over, exit; read back by fp8_debug_trace
__device__ unsigned long long g_trace[8 * 1024];
__device__ unsigned g_trace_n;
#endif

__device__ __forceinline__ void epilogue_warps_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

constexpr int kDecodeMaxStages = 32;
constexpr int kDecodeHeader = 1024;   // barriers, tensor-memory slot and abort flag in front of the stages
constexpr int kDecodeSmemBudget = 225 * 1024;   // header + stages, with the slack for aligning the base

__global__ void __launch_bounds__(kGemmThreads, 1)
decode_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t bar_base = smem_u32(smem);
    const uint32_t stage_base = bar_base + kDecodeHeader;
    const int stages = p.dec_stages, bn = p.dec_bn;
    const uint32_t stage_bytes = (uint32_t)p.dec_a_bytes + (uint32_t)bn * kBK;
    // First column of tile n.  The last tile of a ragged N is moved back to end at N (it recomputes a few columns of
    // its neighbour, same values): a box that hangs over the end of the tensor is filled in slowly, and the CTA
    // that owns it finishes long after the others.
    auto tile_col = [&](int n_blk) { return min(n_blk * bn, max(p.N - bn, 0)); };
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kDecodeMaxStages + s); };
    auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * kDecodeMaxStages + b); };
    auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * kDecodeMaxStages + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + (2 * kDecodeMaxStages + 4) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const uint32_t a_ready_bar = bar_base + 8u * (2 * kDecodeMaxStages + 6);   // fused quantisation: the bytes of A exist
    int *s_bias_x = reinterpret_cast<int *>(smem + (2 * kDecodeMaxStages + 8) * 8);   // ... and their bias
    uint32_t *s_max = reinterpret_cast<uint32_t *>(s_bias_x + 1);                     // five words of the amax reduction
    constexpr uint32_t kCols = 512;   // two accumulators of up to 256 columns

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef FP8LIN_EXPERIMENTS
    __shared__ unsigned trace_slot;
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        trace_slot = atomicAdd(&g_trace_n, 1u) % 1024u;
        g_trace[8 * trace_slot] = global_timer_ns();
    }
#endif
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 4); }
        mbar_init(a_ready_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // whatever follows in the stream (the finalize kernel of a split launch, the next small cast) may take its places
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int num_items = p.tiles_n * p.splits;
    if (warp == 0) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
            // every B byte is read once, every A byte by every CTA: B leaves L2 first, A stays
            const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
            // Ahead of the dependency wait (the launch before this one is the small cast of the activation).  Where the
            // caller vouches that the weight bytes were final before that launch began (inference on weights quantised
            // once), the first ring of B tiles is loaded outright and two more rings are pulled towards L2: the weights
            // stream while the launch before drains and the cast runs.  Otherwise the first ring is only pulled towards
            // L2, which holds no stale data whoever writes those bytes.
            const uint32_t tx_bytes = (uint32_t)p.a_box_bytes + (uint32_t)bn * kBK, a_bytes = (uint32_t)p.dec_a_bytes;
            int early = 0;   // stages whose B tile is already on its way when the loop below starts
            if ((int)blockIdx.x < num_items) {
                const int n_blk = (int)blockIdx.x / p.splits, split0 = (int)blockIdx.x % p.splits;
                const int k0 = split0 * p.kb_per_split, k1 = min(p.num_k, k0 + p.kb_per_split);
                int k = k0 + first_kblock(0, n_blk, k1 - k0);
                const int ring = min(k1 - k0, stages);
                if (p.early_b) {
                    for (int i = 0; i < ring; ++i, k = (k + 1 == k1) ? k0 : k + 1) {
                        mbar_expect_tx(full_bar(i), tx_bytes);
                        tma_load_2d_hint(stage_base + i * stage_bytes + a_bytes, &map_b, full_bar(i), k * kBK, tile_col(n_blk), drop);
                    }
                    early = ring;
                    for (int i = ring; i < min(k1 - k0, p.early_rings * stages); ++i, k = (k + 1 == k1) ? k0 : k + 1)
                        tma_prefetch_l2_2d(&map_b, k * kBK, tile_col(n_blk));
                } else {
                    for (int i = 0; i < ring; ++i, k = (k + 1 == k1) ? k0 : k + 1)
                        tma_prefetch_l2_2d(&map_b, k * kBK, tile_col(n_blk));
                }
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef FP8LIN_EXPERIMENTS
            if (blockIdx.x == 0) g_trace[8 * trace_slot + 1] = global_timer_ns();
#endif
            // One thread runs this loop and its latency is the ceiling of what a CTA can stream (a division per k-block
            // was measured to hold a CTA at 0.25 us per k-block with no loads at all): stage index, phase and
            // addresses advance by increments.
            int s = 0;
            uint32_t ph = 0, full = full_bar(0), empty = empty_bar(0), a_dst = stage_base;
            bool alive = true;
            if (p.qx) {   // the bytes of A are written by this very CTA's epilogue warps: wait until all of them are
                alive = mbar_wait(a_ready_bar, 0u, abort_flag, p.d_status);
                asm volatile("fence.proxy.async.global;" ::: "memory");   // written through the generic proxy, read by TMA
            }
#ifdef FP8LIN_EXPERIMENTS
            if (blockIdx.x == 0) g_trace[8 * trace_slot + 3] = global_timer_ns();
#endif
            for (int item = blockIdx.x; alive && item < num_items; item += gridDim.x) {
                const int n_blk = item / p.splits, split = item % p.splits;
                const int k0 = split * p.kb_per_split, k1 = min(p.num_k, k0 + p.kb_per_split);
                const int b_row = tile_col(n_blk);
                // the k-blocks are walked in a rotated order that differs from tile to tile, so that the CTAs do not
                // all ask L2 for the same few lines of A at the same time
                int k = k0 + first_kblock(0, n_blk, k1 - k0);
                for (int i = k1 - k0; i > 0; --i) {
                    if (!mbar_wait(empty, ph ^ 1u, abort_flag, p.d_status)) { alive = false; break; }
#ifdef FP8LIN_EXPERIMENTS
                    if (p.dbg == 5) mbar_arrive(full);   // timing only: no loads
                    else
#endif
                    if (early > 0) {   // announced and half loaded before the dependency wait
                        --early;
                        tma_load_2d_hint(a_dst, &map_a, full, k * kBK, 0, keep);
                    } else {
                        mbar_expect_tx(full, tx_bytes);
                        tma_load_2d_hint(a_dst, &map_a, full, k * kBK, 0, keep);
                        tma_load_2d_hint(a_dst + a_bytes, &map_b, full, k * kBK, b_row, drop);
                    }
                    k = (k + 1 == k1) ? k0 : k + 1;
                    if (++s == stages) {
                        s = 0; ph ^= 1u; full = full_bar(0); empty = empty_bar(0); a_dst = stage_base;
                    } else {
                        full += 8u; empty += 8u; a_dst += stage_bytes;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t t = 0;
            bool alive = true;
            // the bounded waits below start counting only once the launch before this one has completed
            asm volatile("griddepcontrol.wait;" ::: "memory");
            const uint64_t desc0 = smem_desc_k128(0);   // everything but the address field
            const uint32_t a_step = stage_bytes >> 4, b_off = (uint32_t)p.dec_a_bytes >> 4;
            int s = 0;
            uint32_t ph = 0, full = full_bar(0), empty = empty_bar(0), a16 = stage_base >> 4;   // addresses in 16-byte units
            for (int item = blockIdx.x; alive && item < num_items; item += gridDim.x, ++t) {
                const int split = item % p.splits;
                const int k0 = split * p.kb_per_split, k1 = min(p.num_k, k0 + p.kb_per_split);
                const int buf = t & 1;
                const uint32_t acc_ph = (t >> 1) & 1u;
                if (!mbar_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, p.d_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 256;
                uint32_t accumulate = 0;
                for (int i = k1 - k0; i > 0; --i) {
                    if (!mbar_wait(full, ph, abort_flag, p.d_status)) { alive = false; break; }
                    tc_fence_after();
#ifdef FP8LIN_EXPERIMENTS
                    if (p.dbg == 1 || p.dbg == 5) mbar_arrive(empty);   // timing only: no MMA at all
                    else
#endif
                    {
                        const uint64_t da = desc0 | (uint64_t)a16, db = desc0 | (uint64_t)(a16 + b_off);
#pragma unroll
                        for (int j = 0; j < kBK / kUmmaK; ++j) {   // 32 bytes along a 128-byte row per instruction
                            umma_f8(d_tmem, da + 2u * j, db + 2u * j, p.idesc, accumulate);
                            accumulate = 1u;
                        }
                        umma_commit(empty);
                    }
                    if (++s == stages) {
                        s = 0; ph ^= 1u; full = full_bar(0); empty = empty_bar(0); a16 = stage_base >> 4;
                    } else {
                        full += 8u; empty += 8u; a16 += a_step;
                    }
                }
                if (alive) umma_commit(acc_full_bar(buf));
            }
        }
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the biases may come from the launch before this one
        const int q = warp & 3;  // TMEM lane quarter this warp may address
        int bias_x;
        if (p.qx) {
            // FP8-AMAX of the whole activation by the 128 threads of these warps, in 16-byte vectors
            const int tid = (int)threadIdx.x - 64;
            const int64_t v0 = 0, v1 = (int64_t)p.M * p.K / 8;
            // eight loads in flight per thread at a time: one after the other they cost a trip to L2 each (measured:
            // 5 us for 16 KB, 14 us for 56 KB)
            constexpr int kBatch = 8;
            uint32_t acc = 0;
            for (int64_t base = v0 + tid; base < v1; base += 128 * kBatch) {
                uint4 v[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int64_t i = base + 128 * j;
                    v[j] = i < v1 ? __ldcg(p.qx + i) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    acc = __vmaxu2(acc, v[j].x & 0x7FFF7FFFu);
                    acc = __vmaxu2(acc, v[j].y & 0x7FFF7FFFu);
                    acc = __vmaxu2(acc, v[j].z & 0x7FFF7FFFu);
                    acc = __vmaxu2(acc, v[j].w & 0x7FFF7FFFu);
                }
            }
            uint32_t m = __reduce_max_sync(0xFFFFFFFFu, max(acc & 0xFFFFu, acc >> 16));
            if (lane == 0) s_max[q] = m;
            epilogue_warps_sync();
            const uint32_t fbits = max(max(s_max[0], s_max[1]), max(s_max[2], s_max[3])) << 16;   // bf16 bits of the amax, as a float
            unsigned flags = 0;
            bias_x = bias_from_amax_bits(fbits, FP8_E4, p.q_conv, p.q_margin, &flags);
            if (blockIdx.x == 0 && tid == 0) {
                *p.q_amax = __uint_as_float(fbits);
                *p.q_bias = bias_x;
                if (flags) atomicOr(p.d_status, flags);
            }
            const Pow2Pair p2 = make_pow2_pair(bias_x + format_delta(FP8_E4, p.q_conv));
            bool sat = false;
            for (int64_t base = v0 + tid; base < v1; base += 128 * kBatch) {
                uint4 v[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int64_t i = base + 128 * j;
                    v[j] = i < v1 ? __ldcg(p.qx + i) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int64_t i = base + 128 * j;
                    if (i >= v1) continue;
                    const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
                    uint2 o;
                    o.x = cast4w<FP8_E4, FP8_BF16, true>(w, p2, sat);
                    o.y = cast4w<FP8_E4, FP8_BF16, true>(w + 2, p2, sat);
                    *reinterpret_cast<uint2 *>(p.qx8 + i * 8) = o;
                }
            }
            if (__any_sync(0xFFFFFFFFu, sat) && lane == 0) atomicOr(p.d_status, (unsigned)FP8_FLAG_SATURATED);
            asm volatile("fence.proxy.async.global;" ::: "memory");   // the bytes are read back by this CTA's TMA loads
            __threadfence();
            epilogue_warps_sync();
            if (tid == 0) {
                *s_bias_x = bias_x;
                mbar_arrive(a_ready_bar);
            }
        } else {
            bias_x = __ldcg(p.d_sa);
        }
        const int e = -(bias_x + __ldcg(p.d_sb) + p.delta_sum);
        const Pow2Pair sc = make_pow2_pair(e), sc_one = make_pow2_pair(0);
        const bool two_step = (e < -126 || e > 127);
        uint32_t amax_bits = 0, t = 0;
        GemmParams pp = p;   // what store_direct sees: the tile's own column range, the partial-sum plane of a split
        if (p.splits > 1) {
            pp.out_dt = FP8_F32;
            pp.bias_vec = nullptr;
            pp.d_amax_bits = nullptr;
            pp.vec_ok = (p.N % 4) == 0;
        }
        for (int item = blockIdx.x; item < num_items; item += gridDim.x, ++t) {
            const int n_blk = item / p.splits, split = item % p.splits;
            if (p.splits > 1) pp.out = p.partial + (int64_t)split * p.M * p.N;
            const int col_base = tile_col(n_blk);
            pp.N = min(p.N, col_base + bn);   // columns beyond the tile belong to the next one ...
            pp.col_lo = n_blk * bn;           // ... and those a moved-back last tile recomputes, to the one before
            const int buf = t & 1;
            const uint32_t acc_ph = (t >> 1) & 1u;
            const bool ready = mbar_wait(acc_full_bar(buf), acc_ph, abort_flag, p.d_status);
            if (!__all_sync(0xFFFFFFFFu, ready)) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + buf * 256;
#ifdef FP8LIN_EXPERIMENTS
            if (blockIdx.x == 0 && warp == 2 && lane == 0 && t == 0) g_trace[8 * trace_slot + 4] = global_timer_ns();
#endif
            if (p.dec_cluster > 1) break;   // the accumulator stays where it is for the exchange below
            if (q * 32 < p.M) {   // a warp none of whose rows exists reads nothing
#pragma unroll 1
                for (int c = 0; c < bn; c += 32) {
                    uint32_t r[32];
                    tmem_ld_x32(t_row + c, r);
                    tmem_ld_wait();
                    store_direct(r, q * 32 + lane, col_base + c, pp, p.splits > 1 ? sc_one : sc,
                                 p.splits > 1 ? false : two_step, amax_bits);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(buf));
        }
        if (p.d_amax_bits && p.splits == 1 && p.dec_cluster <= 1) {
            amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
            if (lane == 0 && amax_bits) atomicMax(p.d_amax_bits, amax_bits);
        }
    }

    __syncwarp();  // the single-lane roles rejoin their warps before the block-wide barrier
    if (p.dec_cluster > 1) {
        // Every CTA of the cluster holds the sum over its slice of the contraction in accumulator 0 (its epilogue warps
        // have seen "accumulator full", or given up).  Rank r writes rows [0, M) of it to plane r of a buffer at the
        // start of the leader's stages, [plane][row][bn + 4 floats], and the leader adds the planes in rank order.  With
        // up to eight rows its 128 epilogue threads share the columns, four each (a row per lane would leave the whole
        // tile to a few threads: measured 2 to 4 us per launch at one row); with more rows each lane keeps its own row
        // (its accumulator stays in tensor memory; the column-sharing loop, about a hundred dependent instructions
        // per four outputs on four warps, took 8 us at 64 rows).
        const uint32_t rank = cluster_ctarank();
        const int q = warp & 3, row = q * 32 + lane;
        const bool epi = warp >= 2, share_columns = p.M <= 8;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t row_floats = (uint32_t)bn + 4u;   // padded: the lanes of a warp write 32 different rows at once
        const uint32_t plane_bytes = (uint32_t)p.M * row_floats * 4u;
        cluster_sync_all();   // all slices summed; the leader's stages are no longer read or written
        if (epi && q * 32 < p.M && !*abort_flag && (rank != 0 || share_columns)) {
            const uint32_t dst_row = map_to_cta(stage_base, 0) + rank * plane_bytes + (uint32_t)row * row_floats * 4u;
#pragma unroll 1
            for (int c = 0; c < bn; c += 32) {
                uint32_t r[32];
                tmem_ld_x32(t_row + c, r);
                tmem_ld_wait();
                if (row < p.M) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (c + 4 * j < bn)
                            asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst_row + (uint32_t)(c + 4 * j) * 4u),
                                         "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3]) : "memory");
                }
            }
        }
        cluster_sync_all();   // the planes are written (release / acquire across the cluster)
#ifdef FP8LIN_EXPERIMENTS
        if (blockIdx.x == 0 && threadIdx.x == 64) g_trace[8 * trace_slot + 5] = global_timer_ns();
#endif
        if (epi && rank == 0 && !*abort_flag && !share_columns && q * 32 < p.M) {
            const int e = -((p.qx ? *s_bias_x : __ldcg(p.d_sa)) + __ldcg(p.d_sb) + p.delta_sum);
            const Pow2Pair sc = make_pow2_pair(e);
            const bool two_step = (e < -126 || e > 127);
            const int n_blk = (int)blockIdx.x / p.splits;
            GemmParams pp = p;
            const int col_base = tile_col(n_blk);
            pp.N = min(p.N, col_base + bn);
            pp.col_lo = n_blk * bn;
            uint32_t amax_bits = 0;
            const uint32_t src_row = stage_base + (uint32_t)row * row_floats * 4u;
#pragma unroll 1
            for (int c = 0; c < bn; c += 32) {
                uint32_t r[32];
                tmem_ld_x32(t_row + c, r);
                tmem_ld_wait();
                if (row < p.M) {
                    for (int pl = 1; pl < p.dec_cluster; ++pl) {   // rank order: the sum does not depend on timing
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            if (c + 4 * j < bn) {
                                float4 v;
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                             : "r"(src_row + (uint32_t)pl * plane_bytes + (uint32_t)(c + 4 * j) * 4u));
                                r[4 * j] = __float_as_uint(__uint_as_float(r[4 * j]) + v.x);
                                r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + v.y);
                                r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + v.z);
                                r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + v.w);
                            }
                        }
                    }
                }
                store_direct(r, row, col_base + c, pp, sc, two_step, amax_bits);
            }
            if (p.d_amax_bits) {
                amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
                if (lane == 0 && amax_bits) atomicMax(p.d_amax_bits, amax_bits);
            }
        }
        if (epi && rank == 0 && !*abort_flag && share_columns) {
            const int e = -((p.qx ? *s_bias_x : __ldcg(p.d_sa)) + __ldcg(p.d_sb) + p.delta_sum);
            const Pow2Pair sc = make_pow2_pair(e);
            const bool two_step = (e < -126 || e > 127);
            const int n_blk = (int)blockIdx.x / p.splits;
            const int col_base = tile_col(n_blk), col_lo = n_blk * bn, col_hi = min(p.N, col_base + bn);
            const int quads = bn >> 2;                 // groups of four columns per row
            uint32_t amax_bits = 0;
            // ordinary loads (written by other CTAs before the cluster barrier above): the compiler may overlap iterations
            const float *planes = reinterpret_cast<const float *>(smem + kDecodeHeader);
            const uint32_t plane_floats = plane_bytes >> 2;
#pragma unroll 2
            for (int idx = (int)threadIdx.x - 64; idx < p.M * quads; idx += 128) {
                const int r_out = idx / quads, c4 = (idx - r_out * quads) << 2, col = col_base + c4;
                const float *src = planes + (uint32_t)r_out * row_floats + (uint32_t)c4;
                const float4 first = *reinterpret_cast<const float4 *>(src);
                float v[4] = {first.x, first.y, first.z, first.w};
                for (int pl = 1; pl < p.dec_cluster; ++pl) {   // rank order: the sum does not depend on timing
                    const float4 u = *reinterpret_cast<const float4 *>(src + (uint32_t)pl * plane_floats);
                    v[0] += u.x; v[1] += u.y; v[2] += u.z; v[3] += u.w;
                }
                if (col >= col_hi || col + 4 <= col_lo) continue;
                uint32_t bits[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[i] *= sc.first;
                    if (two_step) v[i] *= sc.second;
                    if (p.bias_vec && col + i < p.N)
                        v[i] += p.bias_dt == FP8_F32 ? __ldg(reinterpret_cast<const float *>(p.bias_vec) + col + i)
                                                     : __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t *>(p.bias_vec) + col + i) << 16);
                    if (p.out_dt == FP8_BF16) {
                        uint32_t w;
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(0.0f), "f"(v[i]));
                        bits[i] = w & 0xFFFFu;
                    } else {
                        bits[i] = __float_as_uint(v[i]);
                    }
                }
                const bool whole = col >= col_lo && col + 4 <= col_hi && p.vec_ok;
                if (p.out_dt == FP8_BF16) {
                    uint16_t *dst = reinterpret_cast<uint16_t *>(p.out) + (int64_t)r_out * p.ldo + col;
                    if (whole) *reinterpret_cast<uint2 *>(dst) = make_uint2(bits[0] | (bits[1] << 16), bits[2] | (bits[3] << 16));
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (col + i < col_lo || col + i >= col_hi) continue;
                        if (!whole) dst[i] = (uint16_t)bits[i];
                        amax_bits = max(amax_bits, (bits[i] & 0x7FFFu) << 16);
                    }
                } else {
                    float *dst = reinterpret_cast<float *>(p.out) + (int64_t)r_out * p.ldo + col;
                    if (whole) *reinterpret_cast<uint4 *>(dst) = make_uint4(bits[0], bits[1], bits[2], bits[3]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (col + i < col_lo || col + i >= col_hi) continue;
                        if (!whole) dst[i] = __uint_as_float(bits[i]);
                        amax_bits = max(amax_bits, bits[i] & 0x7FFFFFFFu);
                    }
                }
            }
            if (p.d_amax_bits) {
                amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
                if (lane == 0 && amax_bits) atomicMax(p.d_amax_bits, amax_bits);
            }
#ifdef FP8LIN_EXPERIMENTS
            if (blockIdx.x == 0 && threadIdx.x == 64) g_trace[8 * trace_slot + 6] = global_timer_ns();
#endif
        }
    }
    if (*abort_flag) __nanosleep(20000);  // let copies and MMAs already issued drain before the memory is released
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, kCols);
#ifdef FP8LIN_EXPERIMENTS
    if (threadIdx.x == 0 && blockIdx.x == 0) g_trace[8 * trace_slot + 2] = global_timer_ns();
#endif
}


// ---------------------------------------------------------------------------
// CTA-pair kernel (cta_group::2)
// ---------------------------------------------------------------------------
//
// Two CTAs of a cluster share one 256x256 output tile.  Each loads its own 128
// rows of A and its own 128 of the 256 B rows (so a stage is 32 KB per CTA and
// the shared-memory pipe carries 64 B/clk of MMA reads plus 64 B/clk of TMA
// writes instead of 96 + 96); the leader CTA's MMA thread issues
// tcgen05.mma.cta_group::2 (M=256, N=256, K=32), which reads both CTAs' shared
// memory and writes each CTA's 128 accumulator rows into that CTA's TMEM.
//
// Signalling: the "stage full" barrier lives in the leader and takes one
// arrive.expect_tx from the leader's producer for the bytes of all four TMA
// loads (the peer's loads name the leader's barrier, which cta_group::2 loads
// may do); "stage empty" and "accumulator full" are tcgen05.commit multicast to
// the same barrier offset in both CTAs; "accumulator empty" lives in the leader
// and collects one arrival per epilogue warp of both CTAs.  None of the loads
// is a multicast load.

#ifndef FP8LIN_PAIR_STAGES
#define FP8LIN_PAIR_STAGES 6
#endif
constexpr int kPairStages = FP8LIN_PAIR_STAGES;
constexpr int kPairBN = 256;       // N of the pair tile (and of the instruction)
constexpr int kPairHalfN = 128;    // B rows each CTA loads

constexpr int kPairStagesAct = 5;  // the kernels with a second output trade one stage for two more slabs per warp

// NHALF = 1: the 256 x 256 pair tile, two accumulators in tensor memory (the epilogue of one tile overlaps the main
// loop of the next).  NHALF = 2: a 256 x 512 pair tile held as ONE accumulator of two 256-column halves: each CTA
// loads its 128 rows of A once per k-block and 2 x 128 rows of B, 48 KB for twice the multiply-adds of the 32 KB
// of the narrow tile -- three quarters of the bytes that cross from L2 into shared memory per FLOP.
template <int STAGES, int SLABS, int NHALF = 1>
struct PairSmemT {
    static constexpr int kStages = STAGES;
    static constexpr int kSlabs = SLABS;
    static constexpr int kABytes = kBM * kBK;
    static constexpr int kBBytes = NHALF * kPairHalfN * kBK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kEpiOffset = STAGES * kStageBytes;
    static constexpr int kBarOffset = kEpiOffset + 4 * SLABS * kSlabBytes;
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kTotal = kBarOffset + kNumBars * 8 + 16;
    static constexpr int kDynamic = kTotal + 1024;
    static constexpr int kTmemCols = 512;
};
using PairSmem = PairSmemT<kPairStages, kPairSlabs>;
using PairSmemAct = PairSmemT<kPairStagesAct, kActSlabs>;
constexpr int kWideStages = 4;
using PairSmemWide = PairSmemT<kWideStages, kPairSlabs, 2>;

// arrive (+ expected bytes) on a barrier addressed in the cluster window
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// TMA load whose completion bytes may be counted on the pair leader's barrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t cluster_bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void umma_f8_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on the barrier at this offset in both CTAs of the pair once all MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3)
        : "memory");
}

__host__ __device__ inline uint32_t make_idesc_pair(int a_fmt, int b_fmt)
{
    return (1u << 4) | ((uint32_t)a_fmt << 7) | ((uint32_t)b_fmt << 10) | ((uint32_t)(kPairBN >> 3) << 17) |
           ((uint32_t)(256 >> 4) << 24);
}

// tiles here are 256 x (256 * NHALF); p.tiles_m / p.tiles_n count those
template <int ACT, int NHALF = 1>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_out2,
                 const GemmParams p)
{
    static_assert(NHALF == 1 || ACT == 0, "the wide tile carries the plain epilogue only");
    using L = PairSmemT<NHALF == 2 ? kWideStages : (ACT ? kPairStagesAct : kPairStages), ACT ? kActSlabs : kPairSlabs, NHALF>;
    constexpr int kStagesL = L::kStages;
    constexpr int kTileN = kPairBN * NHALF;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStagesL + s); };
    auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * kStagesL + b); };
    auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * kStagesL + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOffset + L::kNumBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    // an item is one output tile, or one slice of its contraction when the launch splits it (few tiles, long
    // contraction: partial sums go to the FP32 workspace and splitk_finalize_kernel adds them up)
    const int num_tiles = p.tiles_m * p.tiles_n * p.splits;
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesL; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)L::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    if (p.no_loads) {
        // the stages keep one fixed pattern for the whole run: finite E4M3 bytes of magnitude below 2
        uint32_t *w = reinterpret_cast<uint32_t *>(smem);
        for (int i = threadIdx.x; i < kStagesL * L::kStageBytes / 4; i += kGemmThreads)
            w[i] = ((uint32_t)i * 2654435761u + 0x9E3779B9u * (rank + 1u)) & 0xBFBFBFBFu;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (p.splits > 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the finalize kernel may take its places

    if (warp == 0) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
            uint32_t it = 0, t = 0;
            bool alive = true;
            const uint32_t leader_full0 = map_to_cta(full_bar(0), 0);
            // launched as a programmatic dependent of the cast before it: set-up above overlaps that grid's tail,
            // its bytes are not requested before it has completed
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int tile = pair_id; alive && tile < num_tiles; tile += num_pairs, ++t) {
                int m_blk, n_blk;
                tile_coords(tile / p.splits, p, m_blk, n_blk);
                const int k0 = (tile % p.splits) * p.kb_per_split, k1 = min(p.num_k, k0 + p.kb_per_split);
                // Every other tile of a pair walks the contraction backwards.  All pairs pass from one tile to the
                // next at about the same time, and the next tiles share operand strips with the last ones; what L2
                // still holds of those strips is their far end, which a forward walk would reach last (and evict
                // on the way there).
                const bool backwards = (t & 1u) != 0 && p.serpentine;
                for (int k = k0; k < k1; ++k, ++it) {
                    const int kc = (backwards ? k0 + k1 - 1 - k : k) * kBK;
                    const int s = it % kStagesL;
                    const uint32_t leader_full = leader_full0 + 8u * s;
                    const uint32_t ph = (it / kStagesL) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.d_status)) { alive = false; break; }
                    if (p.no_loads) {   // the stage is "full" as it stands
                        if (rank == 0) mbar_arrive(full_bar(s));
                        continue;
                    }
#ifdef FP8LIN_EXPERIMENTS
                    // timing only (wrong results): every other trip round the ring re-uses what the stages hold, in
                    // whole (11) or for B alone (12) or A alone (13): what fewer bytes from L2 would be worth
                    const bool reuse = ((it / kStagesL) & 1u) != 0;
                    if (reuse && p.dbg == 11) {
                        if (rank == 0) mbar_arrive(full_bar(s));
                        continue;
                    }
                    const bool skip_a = reuse && p.dbg == 13, skip_b = reuse && p.dbg == 12;
                    if (rank == 0) mbar_expect_tx(full_bar(s), skip_a ? 2 * (L::kStageBytes - L::kABytes) : (skip_b ? 2 * L::kABytes : 2 * L::kStageBytes));
#else
                    constexpr bool skip_a = false, skip_b = false;
                    // only the leader arrives, announcing the bytes of all four loads of the pair; the
                    // peer's bytes may land first (the pending arrival keeps the phase open)
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2 * L::kStageBytes);
#endif
                    const uint32_t a_dst = smem_base + s * L::kStageBytes;
                    const int a_row = m_blk * 256 + (int)rank * kBM;
                    if (skip_a) {}
                    else if (p.a_mn) tma_load_2d_pair(a_dst, &map_a, leader_full, a_row, kc);
                    else tma_load_2d_pair(a_dst, &map_a, leader_full, kc, a_row);
#pragma unroll
                    for (int h = 0; h < NHALF && !skip_b; ++h) {   // this CTA's 128 of the 256 B rows of each half of the tile
                        const int b_row = n_blk * kTileN + h * kPairBN + (int)rank * kPairHalfN;
                        const uint32_t b_dst = a_dst + L::kABytes + h * (kPairHalfN * kBK);
                        if (p.b_mn) tma_load_2d_pair(b_dst, &map_b, leader_full, b_row, kc);
                        else tma_load_2d_pair(b_dst, &map_b, leader_full, kc, b_row);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, t = 0;
            bool alive = true;
            // the bounded waits below start counting only once the launch before this one has completed
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int tile = pair_id; alive && tile < num_tiles; tile += num_pairs, ++t) {
                // narrow tile: two accumulators used in turn; wide tile: one accumulator whose two halves are
                // released (and waited for) separately, barrier b standing for half b
                const int buf = NHALF == 2 ? 0 : (t & 1);
                const uint32_t acc_ph = NHALF == 2 ? (t & 1u) : ((t >> 1) & 1u);
                if (!mbar_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, p.d_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kPairBN;
                const int k0 = (tile % p.splits) * p.kb_per_split, k1 = min(p.num_k, k0 + p.kb_per_split);
                auto issue = [&](int s, int k, int h) {
                    const uint32_t a_addr = smem_base + s * L::kStageBytes;
                    const uint32_t b_addr = a_addr + L::kABytes + h * (kPairHalfN * kBK);
                    const uint64_t da = p.a_mn ? smem_desc_mn128(a_addr, 128 * kBK) : smem_desc_k128(a_addr);
                    const uint64_t db = p.b_mn ? smem_desc_mn128(b_addr, 128 * kBK) : smem_desc_k128(b_addr);
                    // per instruction (K = 32): 32 bytes along a 128-byte row, or 32 rows = 4096 bytes
                    const uint32_t step_a = p.a_mn ? 256u : 2u, step_b = p.b_mn ? 256u : 2u;
#pragma unroll
                    for (int j = 0; j < kBK / kUmmaK; ++j)
                        umma_f8_pair(d_tmem + h * kPairBN, da + step_a * j, db + step_b * j, p.idesc, (k > k0 || j > 0) ? 1u : 0u);
                };
                int k = k0;
                if (NHALF == 2) {
                    // The epilogue of the previous tile drains half 0, then half 1.  The first k-blocks of this tile
                    // run on half 0 alone while half 1 is still being read; their stages stay held until half 1 has
                    // used them too.
                    const int ahead = min(k1 - k0, kStagesL - 1);
                    for (int a = 0; alive && a < ahead; ++a) {
                        const uint32_t ia = it + a;
                        if (!mbar_wait(full_bar(ia % kStagesL), (ia / kStagesL) & 1u, abort_flag, p.d_status)) { alive = false; break; }
                        tc_fence_after();
                        issue(ia % kStagesL, k0 + a, 0);
                    }
                    if (alive && !mbar_wait(acc_empty_bar(1), acc_ph ^ 1u, abort_flag, p.d_status)) alive = false;
                    if (!alive) break;
                    tc_fence_after();
                    for (int a = 0; a < ahead; ++a, ++it) {
                        issue(it % kStagesL, k0 + a, 1);
                        umma_commit_pair(empty_bar(it % kStagesL));
                    }
                    k = k0 + ahead;
                }
                for (; k < k1; ++k, ++it) {
                    const int s = it % kStagesL;
                    const uint32_t ph = (it / kStagesL) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.d_status)) { alive = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int h = 0; h < NHALF; ++h) issue(s, k, h);
                    umma_commit_pair(empty_bar(s));
                }
                if (alive) umma_commit_pair(acc_full_bar(buf));
            }
        }
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the biases (and aux) may come from the launch before
        const int q = warp & 3;
        const int e = -(__ldcg(p.d_sa) + __ldcg(p.d_sb) + p.delta_sum);
        const Pow2Pair sc = make_pow2_pair(e);
        const bool two_step = (e < -126 || e > 127);
        uint32_t amax_bits = 0, slab_count = 0;
        const uint32_t warp_slabs = smem_base + L::kEpiOffset + q * L::kSlabs * kSlabBytes;
        const uint32_t leader_acc_empty0 = map_to_cta(acc_empty_bar(0), 0);
        uint32_t t = 0;
        // with a split contraction every item leaves its raw FP32 partial sum in the workspace
        GemmParams pp = p;
        if (p.splits > 1) {
            pp.out_dt = FP8_F32;
            pp.out_stream = 0;   // the partial sums are read back at once
            pp.bias_vec = nullptr;
            pp.d_amax_bits = nullptr;
            pp.tma_out = 0;
            pp.vec_ok = (p.N % 4) == 0;
            pp.ldo = p.N;
        }
        const Pow2Pair sc_one = make_pow2_pair(0);
        for (int tile = pair_id; tile < num_tiles; tile += num_pairs, ++t) {
            int m_blk, n_blk;
            tile_coords(tile / p.splits, p, m_blk, n_blk);
            if (p.splits > 1) pp.out = p.partial + (int64_t)(tile % p.splits) * p.M * p.N;
            const int buf = NHALF == 2 ? 0 : (t & 1);
            const uint32_t acc_ph = NHALF == 2 ? (t & 1u) : ((t >> 1) & 1u);
            const bool ready = mbar_wait(acc_full_bar(buf), acc_ph, abort_flag, p.d_status);
            if (!__all_sync(0xFFFFFFFFu, ready)) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kPairBN;
#pragma unroll 1
            for (int h = 0; h < NHALF; ++h)   // the wide tile: half 0 is handed back to the MMA thread before half 1 is read
                epilogue_tile<kPairBN, ACT, L::kSlabs>(&map_out, &map_out2, t_row + h * kPairBN,
                                                       m_blk * 256 + (int)rank * kBM + q * 32, n_blk * kTileN + h * kPairBN, pp,
                                                       p.splits > 1 ? sc_one : sc, p.splits > 1 ? false : two_step, amax_bits,
                                                       warp_slabs, slab_count,
                                                       leader_acc_empty0 + 8u * (NHALF == 2 ? h : buf), true, lane);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        if (p.d_amax_bits) {
            amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
            if (lane == 0 && amax_bits) atomicMax(p.d_amax_bits, amax_bits);
        }
    }

    __syncwarp();
    if (*abort_flag) __nanosleep(20000);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA releases shared or tensor memory while its peer may still touch it
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)L::kTmemCols)
                     : "memory");
}


// ---------------------------------------------------------------------------
// CTA-pair kernel over a list of independent problems (fp8_linear_group)
// ---------------------------------------------------------------------------
//
// The plain CTA-pair kernel with one more level in its tile loop: the tiles of up to kGroupGemmMax matmuls are
// numbered in one sequence (problem after problem, each in its own rasterisation order) and pair q takes numbers
// q, q + pairs, q + 2 pairs, ...  One launch therefore pays one prologue and one drain for all of them, and the last
// wave of one problem is filled up with the first tiles of the next.  Per tile the three roles look up the problem
// the number falls in (the lists are short and the numbers only grow, so the index only moves forward) and take its
// shapes, layouts, instruction descriptor, tensor maps, biases and output from that entry.  Everything else -- stage
// ring, barriers, accumulator hand-over, epilogue -- is the pair kernel's, and carries on across problem boundaries
// without a pause.  Plain epilogue only, no split contraction.  A tile walks the contraction backwards when its
// number within its own problem falls in an odd round of the pairs, which is the direction the single launch of that
// problem would give it (same sums in the same order: same bits).

constexpr int kGroupGemmMax = 16;

struct GroupGemmParams {
    CUtensorMap map_a[kGroupGemmMax], map_b[kGroupGemmMax], map_out[kGroupGemmMax];
    GemmParams p[kGroupGemmMax];
    int first_tile[kGroupGemmMax + 1];   // tile numbers of problem i: [first_tile[i], first_tile[i + 1])
    int count;
};

template <int NHALF>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_pair_group_kernel(const __grid_constant__ GroupGemmParams gg)
{
    using L = PairSmemT<NHALF == 2 ? kWideStages : kPairStages, kPairSlabs, NHALF>;
    constexpr int kStagesL = L::kStages;
    constexpr int kTileN = kPairBN * NHALF;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStagesL + s); };
    auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * kStagesL + b); };
    auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * kStagesL + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kBarOffset + L::kNumBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int num_tiles = gg.first_tile[gg.count];
    const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    unsigned *const d_status = gg.p[0].d_status;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesL; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)L::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool alive = true;
            const uint32_t leader_full0 = map_to_cta(full_bar(0), 0);
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int pi = 0;
            for (int tile = pair_id; alive && tile < num_tiles; tile += num_pairs) {
                while (tile >= gg.first_tile[pi + 1]) ++pi;
                const GemmParams &p = gg.p[pi];
                const CUtensorMap *map_a = &gg.map_a[pi], *map_b = &gg.map_b[pi];
                const int local = tile - gg.first_tile[pi];
                int m_blk, n_blk;
                tile_coords(local, p, m_blk, n_blk);
                const bool backwards = ((local / num_pairs) & 1) != 0 && p.serpentine;
                for (int k = 0; k < p.num_k; ++k, ++it) {
                    const int kc = (backwards ? p.num_k - 1 - k : k) * kBK;
                    const int s = it % kStagesL;
                    const uint32_t leader_full = leader_full0 + 8u * s;
                    const uint32_t ph = (it / kStagesL) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, d_status)) { alive = false; break; }
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2 * L::kStageBytes);
                    const uint32_t a_dst = smem_base + s * L::kStageBytes;
                    const int a_row = m_blk * 256 + (int)rank * kBM;
                    if (p.a_mn) tma_load_2d_pair(a_dst, map_a, leader_full, a_row, kc);
                    else tma_load_2d_pair(a_dst, map_a, leader_full, kc, a_row);
#pragma unroll
                    for (int h = 0; h < NHALF; ++h) {
                        const int b_row = n_blk * kTileN + h * kPairBN + (int)rank * kPairHalfN;
                        const uint32_t b_dst = a_dst + L::kABytes + h * (kPairHalfN * kBK);
                        if (p.b_mn) tma_load_2d_pair(b_dst, map_b, leader_full, b_row, kc);
                        else tma_load_2d_pair(b_dst, map_b, leader_full, kc, b_row);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, t = 0;
            bool alive = true;
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int pi = 0;
            for (int tile = pair_id; alive && tile < num_tiles; tile += num_pairs, ++t) {
                while (tile >= gg.first_tile[pi + 1]) ++pi;
                const GemmParams &p = gg.p[pi];
                const int buf = NHALF == 2 ? 0 : (t & 1);
                const uint32_t acc_ph = NHALF == 2 ? (t & 1u) : ((t >> 1) & 1u);
                if (!mbar_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, d_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kPairBN;
                const int k1 = p.num_k;
                const uint32_t idesc = p.idesc;
                const bool a_mn = p.a_mn != 0, b_mn = p.b_mn != 0;
                auto issue = [&](int s, int k, int h) {
                    const uint32_t a_addr = smem_base + s * L::kStageBytes;
                    const uint32_t b_addr = a_addr + L::kABytes + h * (kPairHalfN * kBK);
                    const uint64_t da = a_mn ? smem_desc_mn128(a_addr, 128 * kBK) : smem_desc_k128(a_addr);
                    const uint64_t db = b_mn ? smem_desc_mn128(b_addr, 128 * kBK) : smem_desc_k128(b_addr);
                    const uint32_t step_a = a_mn ? 256u : 2u, step_b = b_mn ? 256u : 2u;
#pragma unroll
                    for (int j = 0; j < kBK / kUmmaK; ++j)
                        umma_f8_pair(d_tmem + h * kPairBN, da + step_a * j, db + step_b * j, idesc, (k > 0 || j > 0) ? 1u : 0u);
                };
                int k = 0;
                if (NHALF == 2) {   // as in the pair kernel: the first k-blocks run on half 0 while half 1 is still being read
                    const int ahead = min(k1, kStagesL - 1);
                    for (int a = 0; alive && a < ahead; ++a) {
                        const uint32_t ia = it + a;
                        if (!mbar_wait(full_bar(ia % kStagesL), (ia / kStagesL) & 1u, abort_flag, d_status)) { alive = false; break; }
                        tc_fence_after();
                        issue(ia % kStagesL, a, 0);
                    }
                    if (alive && !mbar_wait(acc_empty_bar(1), acc_ph ^ 1u, abort_flag, d_status)) alive = false;
                    if (!alive) break;
                    tc_fence_after();
                    for (int a = 0; a < ahead; ++a, ++it) {
                        issue(it % kStagesL, a, 1);
                        umma_commit_pair(empty_bar(it % kStagesL));
                    }
                    k = ahead;
                }
                for (; k < k1; ++k, ++it) {
                    const int s = it % kStagesL;
                    const uint32_t ph = (it / kStagesL) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag, d_status)) { alive = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int h = 0; h < NHALF; ++h) issue(s, k, h);
                    umma_commit_pair(empty_bar(s));
                }
                if (alive) umma_commit_pair(acc_full_bar(buf));
            }
        }
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the biases may come from the launch before
        const int q = warp & 3;
        uint32_t amax_bits = 0, slab_count = 0;
        const uint32_t warp_slabs = smem_base + L::kEpiOffset + q * L::kSlabs * kSlabBytes;
        const uint32_t leader_acc_empty0 = map_to_cta(acc_empty_bar(0), 0);
        uint32_t t = 0;
        int pi = 0, cur = -1;
        Pow2Pair sc = make_pow2_pair(0);
        bool two_step = false;
        // the output amax of a problem is folded into its word when this warp moves on to the next problem
        auto flush_amax = [&](int done) {
            if (done >= 0 && gg.p[done].d_amax_bits) {
                amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
                if (lane == 0 && amax_bits) atomicMax(gg.p[done].d_amax_bits, amax_bits);
            }
            amax_bits = 0;
        };
        for (int tile = pair_id; tile < num_tiles; tile += num_pairs, ++t) {
            while (tile >= gg.first_tile[pi + 1]) ++pi;
            const GemmParams &p = gg.p[pi];
            if (pi != cur) {
                flush_amax(cur);
                cur = pi;
                const int e = -(__ldcg(p.d_sa) + __ldcg(p.d_sb) + p.delta_sum);
                sc = make_pow2_pair(e);
                two_step = (e < -126 || e > 127);
            }
            int m_blk, n_blk;
            tile_coords(tile - gg.first_tile[pi], p, m_blk, n_blk);
            const int buf = NHALF == 2 ? 0 : (t & 1);
            const uint32_t acc_ph = NHALF == 2 ? (t & 1u) : ((t >> 1) & 1u);
            const bool ready = mbar_wait(acc_full_bar(buf), acc_ph, abort_flag, d_status);
            if (!__all_sync(0xFFFFFFFFu, ready)) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kPairBN;
#pragma unroll 1
            for (int h = 0; h < NHALF; ++h)
                epilogue_tile<kPairBN, 0, L::kSlabs>(&gg.map_out[pi], &gg.map_out[pi], t_row + h * kPairBN,
                                                     m_blk * 256 + (int)rank * kBM + q * 32, n_blk * kTileN + h * kPairBN, p,
                                                     sc, two_step, amax_bits, warp_slabs, slab_count,
                                                     leader_acc_empty0 + 8u * (NHALF == 2 ? h : buf), true, lane);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        flush_amax(cur);
    }

    __syncwarp();
    if (*abort_flag) __nanosleep(20000);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA releases shared or tensor memory while its peer may still touch it
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)L::kTmemCols)
                     : "memory");
}


// Second half of a split-K matmul: add the partial sums in a fixed order, then
// the same unscale / bias / rounding / amax as the fused epilogue.
// VEC = 4: four adjacent columns per thread through 16-byte loads (N a multiple of 4, output 16-byte aligned), all
// of a thread's partial loads independent and in flight together; VEC = 1: any shape.
template <int VEC>
__global__ void __launch_bounds__(256) splitk_finalize_kernel(const GemmParams p)
{
    // launched as a programmatic dependent of the matmul kernel: nothing of that grid's output is read before this;
    // the launch behind this one may take its places as blocks here retire (it waits the same way)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t total = (int64_t)p.M * p.N;
    // Read at L2, not through the read-only path: the matmul ahead of this launch may itself have written A's bias
    // (activation quantised in the same launch) while this grid was already resident, and a line the read-only path
    // holds on this SM is not refreshed by the dependency wait (seen: the stale word, once in a few launches).
    const int e = -(__ldcg(p.d_sa) + __ldcg(p.d_sb) + p.delta_sum);
    const Pow2Pair sc = make_pow2_pair(e);
    uint32_t amax_bits = 0;
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * VEC; i < total;
         i += (int64_t)gridDim.x * blockDim.x * VEC) {
        float acc[VEC];
#pragma unroll
        for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
#pragma unroll 8
        for (int s = 0; s < p.splits; ++s) {
            const float *src = p.partial + (int64_t)s * total + i;
            if (VEC == 4) {
                const float4 v = __ldcs(reinterpret_cast<const float4 *>(src));
                acc[0] += v.x; acc[1 % VEC] += v.y; acc[2 % VEC] += v.z; acc[3 % VEC] += v.w;
            } else {
                acc[0] += __ldcs(src);
            }
        }
        const int col = (int)(i % p.N);
        uint32_t h[VEC];
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            float v = acc[j] * sc.first * sc.second;
            if (p.bias_vec)
                v += p.bias_dt == FP8_F32
                         ? __ldg(reinterpret_cast<const float *>(p.bias_vec) + col + j)
                         : __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t *>(p.bias_vec) + col + j) << 16);
            if (p.out_dt == FP8_BF16) {
                uint32_t w;
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(0.0f), "f"(v));
                h[j] = w & 0xFFFFu;
                amax_bits = max(amax_bits, (w & 0x7FFFu) << 16);
            } else {
                h[j] = __float_as_uint(v);
                amax_bits = max(amax_bits, h[j] & 0x7FFFFFFFu);
            }
        }
        if (VEC == 4) {
            if (p.out_dt == FP8_BF16)
                *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(p.out) + i) =
                    make_uint2(h[0] | (h[1 % VEC] << 16), h[2 % VEC] | (h[3 % VEC] << 16));
            else
                *reinterpret_cast<uint4 *>(reinterpret_cast<float *>(p.out) + i) =
                    make_uint4(h[0], h[1 % VEC], h[2 % VEC], h[3 % VEC]);
        } else {
            if (p.out_dt == FP8_BF16) reinterpret_cast<uint16_t *>(p.out)[i] = (uint16_t)h[0];
            else reinterpret_cast<float *>(p.out)[i] = __uint_as_float(h[0]);
        }
    }
    if (p.d_amax_bits) {
        amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
        if ((threadIdx.x & 31) == 0 && amax_bits) atomicMax(p.d_amax_bits, amax_bits);
    }
}

// A wait that nothing will ever satisfy, with a caller-chosen (short) limit: exercises the bounded-wait path --
// expiry, sticky flag, orderly return -- without any fault.  One CTA, one mbarrier, no copies.
__global__ void wait_expiry_probe_kernel(unsigned long long limit_ns, unsigned *d_status, unsigned *d_done)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // every thread waits for a phase that no one completes
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, d_status, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0) *d_done = ok ? 2u : 1u;   // 1: the wait gave up and the kernel returned normally
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

constexpr int kBN = 256;
constexpr int kStages = 4;

// Switches of the -DFP8LIN_EXPERIMENTS build (environment variables read once in fp8_create); constants otherwise.
static bool g_force_single = false;  // set from FP8LIN_SINGLE_CTA=1 (A/B comparison of the two kernels)
static int g_group_m = 0;               // set from FP8LIN_GROUP_M (experiments with the tile order)
static bool g_no_splitk = false;        // set from FP8LIN_NO_SPLITK=1
static int g_force_splits = 0;          // set from FP8LIN_SPLITS (experiments with the split count)
static bool g_no_pdl = false;           // set from FP8LIN_NO_PDL=1 (A/B: matmuls launched without programmatic dependence)
static bool g_direct_epilogue = false;  // set from FP8LIN_DIRECT_EPILOGUE=1 (A/B comparison of the epilogues)
constexpr int kDecodeMaxCluster = 8;
static int g_decode_clusters[kDecodeMaxCluster + 1] = {0};   // clusters of each size that can be resident at once
static bool g_no_decode_cluster = false; // set from FP8LIN_DECODE_CLUSTER=0 (A/B: split contractions through global memory only)
static bool g_no_fused_quant = false;    // set from FP8LIN_FUSED_QUANT=0 (A/B: fp8_linear_infer_cast as its two calls)
static int g_early_rings = 2;            // rings of B tiles requested ahead of the dependency wait by fp8_linear_infer (FP8LIN_EARLY_RINGS)
static bool g_no_early_b = false;        // set from FP8LIN_EARLY_B=0 (A/B: fp8_linear_infer without its early weight loads)
static bool g_no_decode_kernel = false; // set from FP8LIN_DECODE_KERNEL=0 (A/B: decode shapes on the fixed-width single-CTA kernel)
static int g_dbg = 0;                   // set from FP8LIN_DECODE_DBG (timing-only variants of the decode kernel)
static int g_force_bn = 0;              // set from FP8LIN_DECODE_BN (experiments with the decode tile width)
static bool g_no_out_stream = false;    // set from FP8LIN_OUT_STREAM=0 (A/B: output stores without the evict-first mark)
static bool g_no_serpentine = false;    // set from FP8LIN_SERPENTINE=0 (A/B: every tile walks the contraction forwards)
static int g_force_wide = -1;           // set from FP8LIN_WIDE=0/1 (A/B: never / always the 256 x 512 pair tile)
static bool g_no_group_gemm = false;    // set from FP8LIN_GROUP_GEMM=0 (A/B: fp8_linear_group as its members' own launches)
static int g_group_order = 0;           // set from FP8LIN_GROUP_ORDER (experiments: 0 shortest contraction first, 1 longest first, 2 as given)
static int g_max_pairs = 0;  // CTA pairs that can be resident at once (0: pair kernel unavailable)

#ifndef FP8LIN_WIDE_DEFAULT
#define FP8LIN_WIDE_DEFAULT 1
#endif
constexpr bool kWideTileDefault = FP8LIN_WIDE_DEFAULT != 0;

constexpr int kStagesF16Acc = 2;  // the FP16-accumulation kind keeps 64 KB of running sums beside its stages
constexpr int kStagesAct = 3;  // single-CTA kernels with a second output: fewer stages, two more slabs per warp

template <int ACT>
static cudaError_t set_smem_attributes()
{
    using LS = GemmSmem<kBN, ACT ? kStagesAct : kStages, ACT ? kActSlabs : kSingleSlabs>;
    using LP = PairSmemT<ACT ? kPairStagesAct : kPairStages, ACT ? kActSlabs : kPairSlabs>;
    cudaError_t e = cudaFuncSetAttribute(gemm_kernel<kBN, ACT ? kStagesAct : kStages, ACT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, LS::kDynamic);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gemm_pair_kernel<ACT>, cudaFuncAttributeMaxDynamicSharedMemorySize, LP::kDynamic);
    if (e == cudaSuccess && ACT == 0)
        e = cudaFuncSetAttribute(gemm_pair_kernel<0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PairSmemWide::kDynamic);

    return e;
}

cudaError_t configure_gemm_kernels(int max_smem_optin)
{
    using L = GemmSmem<kBN, kStages>;
    using LA = GemmSmem<kBN, kStagesAct, kActSlabs>;
    if (L::kDynamic > max_smem_optin || PairSmem::kDynamic > max_smem_optin || LA::kDynamic > max_smem_optin ||
        PairSmemAct::kDynamic > max_smem_optin || PairSmemWide::kDynamic > max_smem_optin ||
        kDecodeSmemBudget + 1024 > max_smem_optin)
        return cudaErrorInvalidValue;
    cudaError_t e = set_smem_attributes<0>();
    if (e == cudaSuccess) e = set_smem_attributes<1>();
    if (e == cudaSuccess) e = set_smem_attributes<2>();
    if (e == cudaSuccess) e = set_smem_attributes<3>();
    if (e == cudaSuccess) e = set_smem_attributes<4>();
    if (e == cudaSuccess) e = set_smem_attributes<5>();
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gemm_kernel<kBN, kStagesF16Acc, 6>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 GemmSmem<kBN, kStagesF16Acc, kActSlabs>::kDynamic);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmemBudget + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gemm_pair_group_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem::kDynamic);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gemm_pair_group_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PairSmemWide::kDynamic);
    if (e != cudaSuccess) return e;
    for (int cs = 2; cs <= kDecodeMaxCluster; ++cs) {   // how many clusters of each size fit the GPU at once
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(cs * 64));
        cfg.blockDim = dim3(kGemmThreads);
        cfg.dynamicSmemBytes = kDecodeSmemBudget + 1024;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, decode_kernel, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        g_decode_clusters[cs] = n;
    }
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return cudaErrorUnknown;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms & ~1), 1, 1);
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = PairSmem::kDynamic;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, gemm_pair_kernel<0>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        clusters = 0;
    }
    g_max_pairs = clusters;
#ifdef FP8LIN_EXPERIMENTS   // A/B switches for measurements; the default build reads no environment variable
    const char *env = getenv("FP8LIN_SINGLE_CTA");
    g_force_single = env && env[0] == '1';
    env = getenv("FP8LIN_GROUP_M");
    g_group_m = env ? atoi(env) : 0;
    env = getenv("FP8LIN_DECODE_CLUSTER");
    g_no_decode_cluster = env && env[0] == '0';
    env = getenv("FP8LIN_FUSED_QUANT");
    g_no_fused_quant = env && env[0] == '0';
    env = getenv("FP8LIN_EARLY_RINGS");
    if (env) g_early_rings = atoi(env);
    env = getenv("FP8LIN_EARLY_B");
    g_no_early_b = env && env[0] == '0';
    env = getenv("FP8LIN_DECODE_KERNEL");
    g_no_decode_kernel = env && env[0] == '0';
    env = getenv("FP8LIN_DECODE_DBG");
    g_dbg = env ? atoi(env) : 0;
    env = getenv("FP8LIN_DECODE_BN");
    g_force_bn = env ? atoi(env) : 0;
    env = getenv("FP8LIN_OUT_STREAM");
    g_no_out_stream = env && env[0] == '0';
    env = getenv("FP8LIN_SERPENTINE");
    g_no_serpentine = env && env[0] == '0';
    env = getenv("FP8LIN_NO_PDL");
    g_no_pdl = env && env[0] == '1';
    env = getenv("FP8LIN_SPLITS");
    g_force_splits = env ? atoi(env) : 0;
    env = getenv("FP8LIN_NO_SPLITK");
    g_no_splitk = env && env[0] == '1';
    env = getenv("FP8LIN_DIRECT_EPILOGUE");
    g_direct_epilogue = env && env[0] == '1';
    env = getenv("FP8LIN_WIDE");
    g_force_wide = env ? atoi(env) : -1;
    env = getenv("FP8LIN_GROUP_GEMM");
    g_no_group_gemm = env && env[0] == '0';
    env = getenv("FP8LIN_GROUP_ORDER");
    g_group_order = env ? atoi(env) : 0;
    if (getenv("FP8LIN_DEBUG")) {
        fprintf(stderr, "fp8lin: %d SMs, %d resident CTA pairs, pair kernel %s\n", sms, clusters, g_force_single ? "off" : "on");
        fprintf(stderr, "fp8lin: resident decode clusters of 2..8 CTAs: %d %d %d %d %d %d %d\n", g_decode_clusters[2],
                g_decode_clusters[3], g_decode_clusters[4], g_decode_clusters[5], g_decode_clusters[6], g_decode_clusters[7],
                g_decode_clusters[8]);
    }
#endif
    return cudaSuccess;
}

// 2-D tensor map over a row-major byte matrix [rows, cols_bytes]: box = box_rows x 128 bytes, 128-byte swizzle.
static bool encode_map(fp8_ctx *ctx, CUtensorMap *map, const void *base, int64_t rows, int64_t cols_bytes,
                       int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols_bytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols_bytes};
    cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box,
                                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Which pair tile a plain matmul takes.  The 256 x 512 tile moves three quarters of the operand bytes per FLOP but
// cannot overlap a tile's epilogue with the next tile's main loop beyond its first k-blocks, and its tiles are
// twice as coarse: it must not add a wave, nor waste much of its width beyond N.
static bool use_wide_tile(int64_t M, int64_t N, int64_t Kc)
{
    if (g_force_wide >= 0) return g_force_wide != 0;
    if (g_max_pairs <= 0) return false;
    const int64_t tm = (M + 255) / 256;
    const int64_t narrow = tm * ((N + 255) / 256), wide_t = tm * ((N + 511) / 512);
    const int64_t waves_n = (narrow + g_max_pairs - 1) / g_max_pairs, waves_w = (wide_t + g_max_pairs - 1) / g_max_pairs;
    const bool no_extra_wave = 2 * waves_w <= waves_n + (waves_n >= 8 ? 1 : 0);
    const bool little_waste = ((N + 511) / 512) * 512 - N <= N / 32;
    return kWideTileDefault && Kc >= 2048 && no_extra_wave && little_waste;
}

// Tile width, split count and stage count of a decode launch, by a time model (microseconds) fitted to measured
// launches of the four layers of a 70B-class decoder block at 1 and 64 rows.  Items (tile, slice of the contraction)
// are dealt round-robin, so the CTAs hold q or q + 1 of them: all stream q items together, then the few with one more
// finish alone.  A CTA streaming among `a` active ones moves bytes at 1 / (1 / solo + a / total): about 42 GB/s each
// with all 148 pulling (6.2 TB/s together), and no more than its own pipeline allows however few remain, which is why
// a last wave with a handful of items costs almost as much as a full one and why the width is chosen to give close
// to a whole number of tiles per SM.  A split contraction adds the finalize launch and the trip of the FP32 partial
// sums to memory and back; every item costs a little set-up.
// The contraction of a tile can also be split across the CTAs of a cluster, which exchange their sums through shared
// memory (no partial sums in global memory, no second launch): one tile per cluster, as many clusters as can be
// resident, the exchange buffer inside the leader's stages.
static void choose_decode(const fp8_ctx *ctx, int64_t M, int64_t N, int num_k, int a_bytes, int *bn_out, int *kb_out,
                          int *stages_out, int *cluster_out)
{
    const int sms = ctx->sm_count;
    const double solo0 = 180e3, total = 8e6;   // bytes per microsecond
    const double finalize_us = 3.5, partial_rate = 3.8e6, item_us = 0.15, exchange_us = 1.0, exchange_rate = 50e3;
    // whatever its width, a k-block costs the two single-thread loops (wait, two loads / wait, four MMAs, commit) this much
    const double kblock_us = 0.36, kOverlapLoss = 0.35;
    const int64_t by_ws = (int64_t)(ctx->partial_bytes / sizeof(float)) / (M * N);
    int64_t cap = num_k / 4 < by_ws ? num_k / 4 : by_ws;
    if (cap > 64) cap = 64;
    if (cap < 1 || g_no_splitk) cap = 1;
    double best = 0;
    *bn_out = 0;
    for (int bn = 32; bn <= 256; bn += 16) {
        const int stage = a_bytes + bn * kBK;
        int stages = (kDecodeSmemBudget - kDecodeHeader - kBM * kBK) / stage;   // 16 KB spare: the A rows read past a stage
        if (stages > kDecodeMaxStages) stages = kDecodeMaxStages;
        if (stages < 3) continue;
        const double in_flight = (double)stages * bn * kBK;
        const double solo = solo0 * (in_flight < 192.0 * 1024 ? in_flight / (192.0 * 1024) : 1.0);
        auto rate = [&](double active) { return 1.0 / (1.0 / solo + active / total); };
        const int64_t tiles = (N + bn - 1) / bn;
        for (int64_t sp = 1; sp <= cap; ++sp) {
            const int64_t kb = (num_k + sp - 1) / sp;
            const int64_t real = (num_k + kb - 1) / kb;
            if (real != sp) continue;
            if (g_force_splits > 0 && real != (g_force_splits < cap ? g_force_splits : cap)) continue;
            if (g_force_bn > 0 && bn != g_force_bn) continue;
            const int64_t items = tiles * real;
            const double item_bytes = (double)kb * bn * kBK;
            const int64_t q = items / sms, extra = items % sms;
            const double floor_us = (double)kb * kblock_us;
            // the two bounds do not hide behind each other completely: the larger plus a share of the smaller
            auto item_time = [&](double active) {
                const double t = item_bytes / rate(active);
                return t > floor_us ? t + kOverlapLoss * floor_us : floor_us + kOverlapLoss * t;
            };
            double cost = q > 0 ? (double)q * item_time((double)sms) : 0.0;
            if (extra > 0) cost += item_time((double)extra);
            cost += item_us * (double)(q + (extra > 0 ? 1 : 0));
            if (bn % 32) cost += 0.3;   // the last half chunk of a tile is stored element by element
            if (real > 1) cost += finalize_us + 8.0 * (double)real * (double)M * (double)N / partial_rate;
            if (*bn_out == 0 || cost < best) {
                best = cost;
                *bn_out = bn;
                *kb_out = (int)kb;
                *stages_out = stages;
                *cluster_out = 1;
            }
        }
        for (int cs = 2; cs <= kDecodeMaxCluster && !g_no_decode_cluster; cs *= 2) {   // 2, 4, 8 (three was measured slower than four)
            const int64_t kb = (num_k + cs - 1) / cs;
            if ((num_k + kb - 1) / kb != cs || kb < 4) continue;
            if (tiles > g_decode_clusters[cs]) continue;
            if ((int64_t)cs * M * (bn + 4) * 4 > (int64_t)stages * stage) continue;   // the exchange buffer (padded rows)
            if (g_force_splits > 0 && cs != g_force_splits) continue;
            if (g_force_bn > 0 && bn != g_force_bn) continue;
            const double item_bytes = (double)kb * bn * kBK;
            const double stream_us = item_bytes / rate((double)(tiles * cs)), floor_us = (double)kb * kblock_us;
            double cost = stream_us > floor_us ? stream_us + kOverlapLoss * floor_us : floor_us + kOverlapLoss * stream_us;
            cost += item_us + exchange_us + (double)(cs - 1) * (double)M * bn * 4.0 / exchange_rate;
            if (bn % 32) cost += 0.3;
            if (*bn_out == 0 || cost < best) {
                best = cost;
                *bn_out = bn;
                *kb_out = (int)kb;
                *stages_out = stages;
                *cluster_out = cs;
            }
        }
    }
    if (*bn_out == 0) {   // nothing matched a forced count: one tile of 256 columns per item, unsplit
        *bn_out = 256;
        *cluster_out = 1;
        *kb_out = num_k;
        *stages_out = (kDecodeSmemBudget - kDecodeHeader - kBM * kBK) / (a_bytes + 256 * kBK);
    }
}

constexpr int64_t kFusedQuantMaxBytes = 64 << 10;
// The activation of a decode launch, to be quantised by that launch itself (decode kernel only).
struct FusedQuant {
    const void *x;     // bf16 [M, Kc], contiguous, 16-byte aligned
    uint8_t *x8;       // out [M, Kc]; run_gemm's `a` must be this buffer
    float *d_amax;     // out
    int32_t *d_bias;   // out; run_gemm's `d_ba` must be this word
    int margin, conv;
};

// Where run_gemm leaves a prepared problem instead of launching it (fp8_linear_group): entry `index` of `gg`, in
// the tile shape the whole group uses.
struct GroupSlot {
    GroupGemmParams *gg;
    int index;
    bool wide;
};

// D[M,N] = A * B^T over a contraction of length Kc, unscaled by 2^-(bias_a + bias_b + delta_sum).
// A is stored [M, Kc] (a_mn = false) or [Kc, M] (a_mn = true); B is stored [N, Kc] or [Kc, N] likewise.
static fp8_status_t run_gemm(fp8_ctx *ctx, const uint8_t *a, int a_fmt, bool a_mn, const int32_t *d_ba,
                             const uint8_t *b, int b_fmt, bool b_mn, const int32_t *d_bb, int delta_sum,
                             const void *bias_vec, int bias_dt, void *out, int out_dt, float *d_amax_out, int64_t M,
                             int64_t N, int64_t Kc, cudaStream_t st, int act = 0, void *out_act = nullptr,
                             const void *aux = nullptr, uint8_t *out8 = nullptr, const int32_t *d_sq = nullptr,
                             int q_fmt = 0, int delta_q = 0, bool no_loads = false, int chunk_kb = 0, bool static_b = false,
                             const FusedQuant *fq = nullptr, GroupSlot *slot = nullptr)
{
    if (M > 0x7FFFFFFF / 2 || N > 0x7FFFFFFF / 2 || Kc > 0x7FFFFFFF / 2) return FP8_ERR_SHAPE;
    const bool pair = g_max_pairs > 0 && M > kBM && !g_force_single && act != 6;
    if (slot && (!pair || act != 0 || no_loads || fq)) return FP8_ERR_UNSUPPORTED;
    CUtensorMap map_a, map_b;
    // an operand stored [Kc, M or N] is fetched as boxes of 128 contraction rows x 128 bytes
    // With a few rows of A (decode) the box covers those rows only, rounded up to the 8-row swizzle atom: the other
    // rows of the stage keep whatever they held and feed output rows that are never stored.  (A 128-row box on a
    // one-row tensor cost 6 us of a 89 us launch, and 59 us for some placements of the activation in memory.)
    const int a_box_rows = (!pair && !a_mn && M < kBM) ? (int)((M + 7) / 8 * 8) : kBM;
    // at most 128 rows, both operands contraction-major, plain epilogue: the decode kernel, tile width chosen here
    const bool decode = !pair && !a_mn && !b_mn && act == 0 && M <= kBM && !g_no_decode_kernel && !no_loads;
    GemmParams p;
    p.dec_bn = p.dec_stages = p.dec_a_bytes = 0;
    p.dec_cluster = 1;
    p.col_lo = 0;
    p.qx = nullptr;
    if (fq) {
        // beyond 64 KB of activation (or outside the decode kernel) the caller quantises with a call of its own
        if (!decode || M * Kc * 2 > kFusedQuantMaxBytes) return FP8_ERR_UNSUPPORTED;
        p.qx = static_cast<const uint4 *>(fq->x);
        p.qx8 = fq->x8;
        p.q_amax = fq->d_amax;
        p.q_bias = fq->d_bias;
        p.q_margin = fq->margin;
        p.q_conv = fq->conv;
    }
    p.early_b = (decode && static_b && !g_no_early_b) ? 1 : 0;
    p.early_rings = g_early_rings;
    p.dbg = g_dbg;
    int dec_kb = 0;
    if (decode) {
        p.dec_a_bytes = a_box_rows * kBK;
        choose_decode(ctx, M, N, (int)((Kc + kBK - 1) / kBK), p.dec_a_bytes, &p.dec_bn, &dec_kb, &p.dec_stages, &p.dec_cluster);
#ifdef FP8LIN_EXPERIMENTS
        if (getenv("FP8LIN_DEBUG"))
            fprintf(stderr, "fp8lin decode M=%lld N=%lld K=%lld: bn %d, %d k-blocks per item, %d stages, cluster %d\n",
                    (long long)M, (long long)N, (long long)Kc, p.dec_bn, dec_kb, p.dec_stages, p.dec_cluster);
#endif
    }
    const bool ok_a = a_mn ? encode_map(ctx, &map_a, a, Kc, M, kBK) : encode_map(ctx, &map_a, a, M, Kc, a_box_rows);
    const bool ok_b = b_mn ? encode_map(ctx, &map_b, b, Kc, N, kBK)
                           : encode_map(ctx, &map_b, b, N, Kc, decode ? p.dec_bn : (pair ? kPairHalfN : kBN));
    if (!ok_a || !ok_b) return FP8_ERR_CUDA;
    p.group_m = g_group_m > 0 ? g_group_m : kGroupM;
    p.serpentine = g_no_serpentine ? 0 : 1;
    p.out_stream = (!g_no_out_stream && (int64_t)M * N * (out_dt == FP8_F32 ? 4 : 2) >= kStreamOutBytes) ? 1 : 0;
    p.a_mn = a_mn ? 1 : 0;
    p.b_mn = b_mn ? 1 : 0;
    p.a_box_bytes = a_box_rows * kBK;
    p.M = (int)M; p.N = (int)N; p.K = (int)Kc;
    const bool wide = pair && act == 0 && (slot ? slot->wide : use_wide_tile(M, N, Kc));
    p.tiles_m = (int)((M + (pair ? 256 : kBM) - 1) / (pair ? 256 : kBM));
    p.tiles_n = (int)((N + (wide ? 2 * kBN : kBN) - 1) / (wide ? 2 * kBN : kBN));
    p.num_k = (int)((Kc + kBK - 1) / kBK);
    if ((int64_t)p.tiles_m * p.tiles_n > 0x7FFFFFFF) return FP8_ERR_SHAPE;
    // Few output tiles and a long contraction (the decode regime): split the contraction so that every SM
    // streams operand bytes; partial sums go through the context's FP32 workspace.
    p.splits = 1;
    p.kb_per_split = p.num_k;
    p.partial = ctx->d_partial;
    if (act == 6) {   // FP16 accumulation: one slice per FP16 addition, all slices of a tile on one CTA
        p.kb_per_split = chunk_kb > 0 ? chunk_kb : 1;
        p.splits = (p.num_k + p.kb_per_split - 1) / p.kb_per_split;
    }
    if (decode) {
        p.tiles_n = (int)((N + p.dec_bn - 1) / p.dec_bn);
        p.kb_per_split = dec_kb;
        p.splits = (p.num_k + dec_kb - 1) / dec_kb;
    }
    if (!pair && !decode && !g_no_splitk && !act) {
        const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
        if (tiles < 2 * ctx->sm_count && p.num_k >= 8) {
            // Pick the split count by a time model of the launch (microseconds), fitted to measured launches of the
            // four decode layers of a 70B-class model at 1 and 64 rows, 1 to 12 splits.  Items are dealt round-robin,
            // so the CTAs hold q or q + 1 items: all stream q items together, then the few with one more finish alone.
            // A CTA streaming among `a` active ones moves bytes at 1 / (1 / solo + a / total): about 42 GB/s each
            // with all 148 pulling (6.2 TB/s together), and no more than its own pipeline allows however few remain
            // (which is why a last wave with a handful of items costs almost as much as a full one).  A split
            // launch adds the finalize kernel and the trip of the FP32 partial sums to memory and back.
            const int64_t by_k = p.num_k / 4;
            const int64_t by_ws = (int64_t)(ctx->partial_bytes / sizeof(float)) / (M * N);
            int64_t cap = by_k < by_ws ? by_k : by_ws;
            if (cap > 64) cap = 64;
            const double sms = (double)ctx->sm_count;
            const double solo = 180e3, total = 8e6;            // bytes per microsecond
            const double finalize_us = 1.0, partial_rate = 3.8e6;
            auto rate = [&](double active) { return 1.0 / (1.0 / solo + active / total); };
            double best = 0;
            int64_t best_kb = p.num_k;
            for (int64_t sp = 1; sp <= cap; ++sp) {
                const int64_t kb = (p.num_k + sp - 1) / sp;
                const int64_t real = (p.num_k + kb - 1) / kb;
                if (real != sp) continue;
                const int64_t items = tiles * real;
                const double item_bytes = (double)kb * kBN * kBK;
                const int64_t q = items / ctx->sm_count, extra = items % ctx->sm_count;
                double cost = q > 0 ? (double)q * item_bytes / rate(sms) : 0.0;
                if (extra > 0) cost += item_bytes / rate((double)extra);
                if (real > 1) cost += finalize_us + 8.0 * (double)real * (double)M * (double)N / partial_rate;
                if (sp == 1 || cost < best) {
                    best = cost;
                    best_kb = kb;
                }
            }
            if (g_force_splits > 0) {   // an experiment's count, still bounded by the workspace
                const int64_t forced = g_force_splits < by_ws ? g_force_splits : (by_ws > 0 ? by_ws : 1);
                best_kb = (p.num_k + forced - 1) / forced;
            }
            p.kb_per_split = (int)best_kb;
            p.splits = (p.num_k + p.kb_per_split - 1) / p.kb_per_split;
        }
    }
    if (pair && !g_no_splitk && !act && !no_loads && !slot) {
        // Fewer tiles than CTA pairs and a long contraction: slice it so that most pairs have work.  The second
        // launch and the trip of the partial sums through memory cost 6-7 us, so a slice keeps at least sixteen
        // k-blocks (measured: 1024 x 1024 x 8192 27 -> 22 us, 512 x 512 x 16384 46 -> 20 us; at 32 k-blocks or fewer
        // per tile the unsplit launch wins); the partial sums must fit the workspace.
        const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
        int64_t sp = g_max_pairs / tiles;
        const int64_t by_k = p.num_k / 16, by_ws = (int64_t)(ctx->partial_bytes / sizeof(float)) / (M * N);
        if (sp > by_k) sp = by_k;
        if (sp > 16) sp = 16;
        if (g_force_splits > 0) sp = g_force_splits;
        if (sp > by_ws) sp = by_ws;   // never beyond the workspace, whatever asked for the count
        if (sp > 1) {
            p.kb_per_split = (int)((p.num_k + sp - 1) / sp);
            p.splits = (p.num_k + p.kb_per_split - 1) / p.kb_per_split;
        }
    }
    p.d_sa = d_ba; p.d_sb = d_bb; p.delta_sum = delta_sum;
    p.bias_vec = bias_vec; p.bias_dt = bias_dt;
    p.out = out; p.out_dt = out_dt; p.ldo = N;
    const int64_t esz = out_dt == FP8_BF16 ? 2 : 4;
    p.vec_ok = ((reinterpret_cast<uintptr_t>(out) & 15u) == 0 && (N * esz) % 16 == 0) ? 1 : 0;
    p.tma_out = (p.vec_ok && !g_direct_epilogue && !decode) ? 1 : 0;
    p.act = act;
    p.aux = aux;
    p.has_out2 = out_act ? 1 : 0;
    p.out8 = out8;
    p.d_sq = d_sq;
    p.q_fmt = q_fmt;
    p.delta_q = delta_q;
    p.no_loads = no_loads ? 1 : 0;
    if (no_loads && !pair) return FP8_ERR_UNSUPPORTED;
    CUtensorMap map_out = map_a;  // placeholder when the staged epilogue is off (never dereferenced then)
    CUtensorMap map_out2 = map_a;
    auto encode_out = [&](CUtensorMap *m, void *base, int64_t cols) {
        cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)M};
        cuuint64_t strides[1] = {(cuuint64_t)(cols * esz)};
        cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32};
        cuuint32_t estr[2] = {1, 1};
        return ctx->encode_tiled(m, esz == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, base,
                                 dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    if (act == 6) {
        p.tma_out = 0;   // the FP16-accumulation kind stores from registers
    } else if (act) {
        // the activated output always goes through the staged epilogue (callers have checked its alignment)
        p.tma_out = 1;
        p.vec_ok = 1;
        // the second tensor is as wide as the output, half as wide (SwiGLU) or twice as wide (its backward)
        const int64_t cols2 = act == 4 ? N / 2 : (act == 5 ? 2 * N : N);
        if (out_act && !encode_out(&map_out2, out_act, cols2)) return FP8_ERR_CUDA;
        if (out && !encode_out(&map_out, out, N)) return FP8_ERR_CUDA;
    } else if (p.tma_out) {
        if (!encode_out(&map_out, out, N)) return FP8_ERR_CUDA;
    }
    p.d_amax_bits = reinterpret_cast<unsigned *>(d_amax_out);
    p.d_status = ctx->d_status;
    p.idesc = (pair ? make_idesc_pair(a_fmt, b_fmt) : make_idesc(a_fmt, b_fmt, decode ? p.dec_bn : kBN)) | ((uint32_t)p.a_mn << 15) |
              ((uint32_t)p.b_mn << 16);
    if (d_amax_out && cudaMemsetAsync(d_amax_out, 0, sizeof(float), st) != cudaSuccess) return FP8_ERR_CUDA;
    if (slot) {   // prepared, not launched: the group's one launch runs it
        GroupGemmParams &g = *slot->gg;
        g.p[slot->index] = p;
        g.map_a[slot->index] = map_a;
        g.map_b[slot->index] = map_b;
        g.map_out[slot->index] = map_out;
        return FP8_OK;
    }
    int tiles = p.tiles_m * p.tiles_n;
    const bool finalize = p.splits > 1 && act != 6 && p.dec_cluster <= 1;
    count_launch(finalize ? 2 : 1);
    if (pair) {
        const int items = tiles * p.splits;
        int pairs = items < g_max_pairs ? items : g_max_pairs;
        const dim3 grid(2 * pairs);
        switch (act) {
        case 1: gemm_pair_kernel<1><<<grid, kGemmThreads, PairSmemAct::kDynamic, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 2: gemm_pair_kernel<2><<<grid, kGemmThreads, PairSmemAct::kDynamic, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 3: gemm_pair_kernel<3><<<grid, kGemmThreads, PairSmemAct::kDynamic, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 4: gemm_pair_kernel<4><<<grid, kGemmThreads, PairSmemAct::kDynamic, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 5: gemm_pair_kernel<5><<<grid, kGemmThreads, PairSmemAct::kDynamic, st>>>(map_a, map_b, map_out, map_out2, p); break;
        default: {
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = grid;
            cfg.blockDim = dim3(kGemmThreads);
            cfg.dynamicSmemBytes = wide ? PairSmemWide::kDynamic : PairSmem::kDynamic;
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            cudaError_t le = wide ? cudaLaunchKernelEx(&cfg, gemm_pair_kernel<0, 2>, map_a, map_b, map_out, map_out2, p)
                                  : cudaLaunchKernelEx(&cfg, gemm_pair_kernel<0>, map_a, map_b, map_out, map_out2, p);
            if (le != cudaSuccess) return FP8_ERR_CUDA;
            break;
        }
        }
    } else if (decode) {
        const int items = p.tiles_n * p.splits;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)p.dec_cluster;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        // a cluster launch has one item per CTA (the clusters fit the GPU at once, by choose_decode)
        cfg.gridDim = dim3((unsigned)(p.dec_cluster > 1 ? items : (items < ctx->sm_count ? items : ctx->sm_count)));
        cfg.blockDim = dim3(kGemmThreads);
        cfg.dynamicSmemBytes = kDecodeSmemBudget + 1024;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = g_no_pdl ? 1 : 2;
        if (cudaLaunchKernelEx(&cfg, decode_kernel, map_a, map_b, p) != cudaSuccess) return FP8_ERR_CUDA;
    } else {
        int items = act == 6 ? tiles : tiles * p.splits;
        int grid = items < ctx->sm_count ? items : ctx->sm_count;
        constexpr int kActDyn = GemmSmem<kBN, kStagesAct, kActSlabs>::kDynamic;
        switch (act) {
        case 6: gemm_kernel<kBN, kStagesF16Acc, 6><<<grid, kGemmThreads, GemmSmem<kBN, kStagesF16Acc, kActSlabs>::kDynamic, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 1: gemm_kernel<kBN, kStagesAct, 1><<<grid, kGemmThreads, kActDyn, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 2: gemm_kernel<kBN, kStagesAct, 2><<<grid, kGemmThreads, kActDyn, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 3: gemm_kernel<kBN, kStagesAct, 3><<<grid, kGemmThreads, kActDyn, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 4: gemm_kernel<kBN, kStagesAct, 4><<<grid, kGemmThreads, kActDyn, st>>>(map_a, map_b, map_out, map_out2, p); break;
        case 5: gemm_kernel<kBN, kStagesAct, 5><<<grid, kGemmThreads, kActDyn, st>>>(map_a, map_b, map_out, map_out2, p); break;
        default: {
            // may start while the launch before it drains (its own first instruction that reads memory waits)
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)grid);
            cfg.blockDim = dim3(kGemmThreads);
            cfg.dynamicSmemBytes = GemmSmem<kBN, kStages>::kDynamic;
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = g_no_pdl ? 0 : 1;
            if (cudaLaunchKernelEx(&cfg, gemm_kernel<kBN, kStages, 0>, map_a, map_b, map_out, map_out2, p) != cudaSuccess)
                return FP8_ERR_CUDA;
            break;
        }
        }
    }
    if (finalize) {
        if (cudaGetLastError() != cudaSuccess) return FP8_ERR_CUDA;
        const bool vec = p.vec_ok && (N % 4) == 0;
        int64_t threads = vec ? M * N / 4 : M * N;
        int64_t blocks = (threads + 255) / 256;
        if (blocks > (int64_t)ctx->sm_count * 16) blocks = (int64_t)ctx->sm_count * 16;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t le = vec ? cudaLaunchKernelEx(&cfg, splitk_finalize_kernel<4>, p)
                             : cudaLaunchKernelEx(&cfg, splitk_finalize_kernel<1>, p);
        if (le != cudaSuccess) return FP8_ERR_CUDA;
    }
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool out_dtype_ok(int dt) { return dt == FP8_BF16 || dt == FP8_F32; }

}  // namespace fp8lin

extern "C" {

static fp8_status_t linear_fwd_impl(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                                    const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y,
                                    fp8_dtype_t y_dt, float *d_amax_y, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                                    void *stream, fp8lin::GroupSlot *slot)
{
    using namespace fp8lin;
    if (!ctx || !x8 || !d_bx || !w8 || !d_bw || !y) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)y_dt < 0 || (int)y_dt > 2 || (int)bias_dt < 0 || (int)bias_dt > 2)
        return FP8_ERR_DTYPE;
    if (!out_dtype_ok(y_dt) || (bias_vec && !out_dtype_ok(bias_dt))) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    if (!aligned16(x8) || !aligned16(w8) || (K % 16) != 0 || (reinterpret_cast<uintptr_t>(y) & 3u)) return FP8_ERR_ALIGN;
    int delta = 2 * format_delta(FP8_E4, conv);
    return run_gemm(ctx, x8, FP8_E4, false, d_bx, w8, FP8_E4, false, d_bw, delta, bias_vec, bias_dt, y, y_dt, d_amax_y,
                    T, N, K, (cudaStream_t)stream, 0, nullptr, nullptr, nullptr, nullptr, 0, 0, false, 0, false, nullptr,
                    slot);
}

fp8_status_t fp8_linear_fwd(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                            const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y,
                            fp8_dtype_t y_dt, float *d_amax_y, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                            void *stream)
{
    return linear_fwd_impl(ctx, x8, d_bx, w8, d_bw, bias_vec, bias_dt, y, y_dt, d_amax_y, T, K, N, conv, stream, nullptr);
}

fp8_status_t fp8_linear_infer(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                              const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y,
                              fp8_dtype_t y_dt, float *d_amax_y, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                              void *stream)
{
    using namespace fp8lin;
    if (!ctx || !x8 || !d_bx || !w8 || !d_bw || !y) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)y_dt < 0 || (int)y_dt > 2 || (int)bias_dt < 0 || (int)bias_dt > 2)
        return FP8_ERR_DTYPE;
    if (!out_dtype_ok(y_dt) || (bias_vec && !out_dtype_ok(bias_dt))) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    if (!aligned16(x8) || !aligned16(w8) || (K % 16) != 0 || (reinterpret_cast<uintptr_t>(y) & 3u)) return FP8_ERR_ALIGN;
    int delta = 2 * format_delta(FP8_E4, conv);
    return run_gemm(ctx, x8, FP8_E4, false, d_bx, w8, FP8_E4, false, d_bw, delta, bias_vec, bias_dt, y, y_dt, d_amax_y,
                    T, N, K, (cudaStream_t)stream, 0, nullptr, nullptr, nullptr, nullptr, 0, 0, false, 0, true);
}

#ifdef FP8LIN_EXPERIMENTS
__attribute__((visibility("default"))) int fp8_debug_trace(unsigned long long *host_out, int clear)
{
    unsigned n = 0;
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(&n, fp8lin::g_trace_n, sizeof(n));
    cudaMemcpyFromSymbol(host_out, fp8lin::g_trace, sizeof(unsigned long long) * 8 * 1024);
    if (clear) {
        unsigned zero = 0;
        cudaMemcpyToSymbol(fp8lin::g_trace_n, &zero, sizeof(zero));
    }
    return (int)n;
}
#endif

fp8_status_t fp8_linear_infer_cast(fp8_ctx *ctx, const void *x, fp8_dtype_t x_dt, int32_t margin, float *d_amax_x,
                                   int32_t *d_bx, uint8_t *x8, const uint8_t *w8, const int32_t *d_bw, const void *bias_vec,
                                   fp8_dtype_t bias_dt, void *y, fp8_dtype_t y_dt, float *d_amax_y, int64_t T, int64_t K,
                                   int64_t N, fp8_conv_t conv, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !x || !d_amax_x || !d_bx || !x8 || !w8 || !d_bw || !y) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)y_dt < 0 || (int)y_dt > 2 || (int)bias_dt < 0 || (int)bias_dt > 2 ||
        (int)x_dt < 0 || (int)x_dt > 2)
        return FP8_ERR_DTYPE;
    if (!out_dtype_ok(y_dt) || (bias_vec && !out_dtype_ok(bias_dt))) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    if (!aligned16(x8) || !aligned16(w8) || (K % 16) != 0 || (reinterpret_cast<uintptr_t>(y) & 3u)) return FP8_ERR_ALIGN;
    const int delta = 2 * format_delta(FP8_E4, conv);
    if (x_dt == FP8_BF16 && aligned16(x) && T <= kBM && g_max_pairs >= 0 && !g_no_fused_quant) {
        const FusedQuant fq = {x, x8, d_amax_x, d_bx, margin, (int)conv};
        const fp8_status_t st = run_gemm(ctx, x8, FP8_E4, false, d_bx, w8, FP8_E4, false, d_bw, delta, bias_vec, bias_dt, y,
                                         y_dt, d_amax_y, T, N, K, (cudaStream_t)stream, 0, nullptr, nullptr, nullptr,
                                         nullptr, 0, 0, false, 0, true, &fq);
        if (st != FP8_ERR_UNSUPPORTED) return st;
    }
    // any other case: the two calls this one stands for
    const fp8_status_t st = fp8_cast_e4(ctx, x, x_dt, T, K, K, nullptr, conv, margin, d_amax_x, d_bx, x8, nullptr, stream);
    if (st != FP8_OK) return st;
    return fp8_linear_infer(ctx, x8, d_bx, w8, d_bw, bias_vec, bias_dt, y, y_dt, d_amax_y, T, K, N, conv, stream);
}

fp8_status_t fp8_selftest_mma_ceiling(fp8_ctx *ctx, void *out, const int32_t *d_zero, int64_t M, int64_t N, int64_t K,
                                      void *stream)
{
    using namespace fp8lin;
    if (!ctx || !out || !d_zero) return FP8_ERR_NULL;
    if (M <= kBM || N <= 0 || K <= 0) return FP8_ERR_SHAPE;
    if (!aligned16(out) || (N % 8) != 0 || (K % 16) != 0) return FP8_ERR_ALIGN;
    // the operand maps are encoded (over the output buffer's address) but never used: no load is issued
    return run_gemm(ctx, static_cast<const uint8_t *>(out), FP8_E4, false, d_zero, static_cast<const uint8_t *>(out),
                    FP8_E4, false, d_zero, 0, nullptr, 0, out, FP8_BF16, nullptr, M, N, K, (cudaStream_t)stream, 0, nullptr,
                    nullptr, nullptr, nullptr, 0, 0, true);
}

fp8_status_t fp8_selftest_wait_expiry(fp8_ctx *ctx, uint64_t limit_ns, void *stream)
{
    using namespace fp8lin;
    if (!ctx) return FP8_ERR_NULL;
    if (limit_ns == 0 || limit_ns > 100ull * 1000ull * 1000ull) return FP8_ERR_SHAPE;   // at most 100 ms
    cudaStream_t st = (cudaStream_t)stream;
    unsigned *done = ctx->d_slots + (kReduceSlots - 1) * kSlotWords + 3;   // a word no reduction reads
    count_launch();
    wait_expiry_probe_kernel<<<1, 64, 0, st>>>((unsigned long long)limit_ns, ctx->d_status, done);
    if (cudaGetLastError() != cudaSuccess) return FP8_ERR_CUDA;
    unsigned host = 0;
    if (cudaMemcpyAsync(&host, done, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(done, 0, sizeof(unsigned), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
        return FP8_ERR_CUDA;
    return host == 1u ? FP8_OK : FP8_ERR_CUDA;
}

fp8_status_t fp8_linear_fwd_act(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                                const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, void *y_pre, void *y_act,
                                fp8_act_t act, float *d_amax_act, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                                void *stream)
{
    using namespace fp8lin;
    if (!ctx || !x8 || !d_bx || !w8 || !d_bw || !y_act) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)bias_dt < 0 || (int)bias_dt > 2 ||
        ((int)act != (int)FP8_ACT_GELU && (int)act != (int)FP8_ACT_SWIGLU))
        return FP8_ERR_DTYPE;
    if (bias_vec && !out_dtype_ok(bias_dt)) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    const bool swiglu = act == FP8_ACT_SWIGLU;
    if (!aligned16(x8) || !aligned16(w8) || (K % 16) != 0 || !aligned16(y_act) || (y_pre && !aligned16(y_pre)) ||
        (N % (swiglu ? 64 : 8)) != 0)
        return FP8_ERR_ALIGN;
    int delta = 2 * format_delta(FP8_E4, conv);
    return run_gemm(ctx, x8, FP8_E4, false, d_bx, w8, FP8_E4, false, d_bw, delta, bias_vec, bias_dt, y_pre, FP8_BF16,
                    d_amax_act, T, N, K, (cudaStream_t)stream, swiglu ? 4 : 1, y_act);
}

static fp8_status_t linear_dgrad_impl(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                                      const uint8_t *w8_t, const int32_t *d_bw, void *dx, fp8_dtype_t dx_dt,
                                      float *d_amax_dx, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream,
                                      fp8lin::GroupSlot *slot)
{
    using namespace fp8lin;
    if (!ctx || !dy8 || !d_bg || (!w8 && !w8_t) || !d_bw || !dx) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)dx_dt < 0 || (int)dx_dt > 2) return FP8_ERR_DTYPE;
    if (!out_dtype_ok(dx_dt)) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    // the transposed copy W8T[K,N] is contracted along contiguous bytes; W8[N,K] itself is read with its K
    // index contiguous and the contraction strided
    const bool w_mn = (w8_t == nullptr);
    const uint8_t *w = w_mn ? w8 : w8_t;
    if (!aligned16(dy8) || !aligned16(w) || (N % 16) != 0 || (w_mn && (K % 16) != 0) ||
        (reinterpret_cast<uintptr_t>(dx) & 3u))
        return FP8_ERR_ALIGN;
    int delta = format_delta(FP8_E5, conv) + format_delta(FP8_E4, conv);
    return run_gemm(ctx, dy8, FP8_E5, false, d_bg, w, FP8_E4, w_mn, d_bw, delta, nullptr, 0, dx, dx_dt, d_amax_dx, T, K,
                    N, (cudaStream_t)stream, 0, nullptr, nullptr, nullptr, nullptr, 0, 0, false, 0, false, nullptr, slot);
}

fp8_status_t fp8_linear_dgrad(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                              const uint8_t *w8_t, const int32_t *d_bw, void *dx, fp8_dtype_t dx_dt,
                              float *d_amax_dx, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream)
{
    return linear_dgrad_impl(ctx, dy8, d_bg, w8, w8_t, d_bw, dx, dx_dt, d_amax_dx, T, K, N, conv, stream, nullptr);
}

fp8_status_t fp8_linear_dgrad_act(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                                  const uint8_t *w8_t, const int32_t *d_bw, const void *y_pre, void *dx, void *dx_act,
                                  fp8_act_t act, float *d_amax_act, int64_t T, int64_t K, int64_t N, fp8_conv_t conv,
                                  void *stream)
{
    using namespace fp8lin;
    if (!ctx || !dy8 || !d_bg || (!w8 && !w8_t) || !d_bw || !y_pre || !dx_act) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || ((int)act != (int)FP8_ACT_GELU && (int)act != (int)FP8_ACT_SWIGLU))
        return FP8_ERR_DTYPE;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    const bool w_mn = (w8_t == nullptr);
    const uint8_t *w = w_mn ? w8 : w8_t;
    const bool swiglu = act == FP8_ACT_SWIGLU;
    if (!aligned16(dy8) || !aligned16(w) || (N % 16) != 0 || (w_mn && (K % 16) != 0) || !aligned16(y_pre) ||
        !aligned16(dx_act) || (dx && !aligned16(dx)) || (K % (swiglu ? 32 : 8)) != 0)
        return FP8_ERR_ALIGN;
    int delta = format_delta(FP8_E5, conv) + format_delta(FP8_E4, conv);
    return run_gemm(ctx, dy8, FP8_E5, false, d_bg, w, FP8_E4, w_mn, d_bw, delta, nullptr, 0, dx, FP8_BF16, d_amax_act, T,
                    K, N, (cudaStream_t)stream, swiglu ? 5 : 2, dx_act, y_pre);
}

fp8_status_t fp8_linear_fwd_q(fp8_ctx *ctx, const uint8_t *x8, const int32_t *d_bx, const uint8_t *w8,
                              const int32_t *d_bw, const void *bias_vec, fp8_dtype_t bias_dt, fp8_act_t act, void *y_pre,
                              void *z, uint8_t *z8, const int32_t *d_bz, float *d_amax_z, int64_t T, int64_t K,
                              int64_t N, fp8_conv_t conv, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !x8 || !d_bx || !w8 || !d_bw || !z8 || !d_bz) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)bias_dt < 0 || (int)bias_dt > 2 || (int)act < (int)FP8_ACT_NONE ||
        (int)act > (int)FP8_ACT_SWIGLU)
        return FP8_ERR_DTYPE;
    if (bias_vec && !out_dtype_ok(bias_dt)) return FP8_ERR_UNSUPPORTED;
    if (act == FP8_ACT_NONE && y_pre) return FP8_ERR_UNSUPPORTED;  // without an activation z is the output itself
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    if (!aligned16(x8) || !aligned16(w8) || (K % 16) != 0 || !aligned16(z8) || (z && !aligned16(z)) ||
        (y_pre && !aligned16(y_pre)) || (N % (act == FP8_ACT_SWIGLU ? 64 : 16)) != 0)
        return FP8_ERR_ALIGN;
    int delta = 2 * format_delta(FP8_E4, conv);
    const int kind = act == FP8_ACT_GELU ? 1 : (act == FP8_ACT_SWIGLU ? 4 : 3);
    return run_gemm(ctx, x8, FP8_E4, false, d_bx, w8, FP8_E4, false, d_bw, delta, bias_vec, bias_dt, y_pre, FP8_BF16,
                    d_amax_z, T, N, K, (cudaStream_t)stream, kind, z, nullptr, z8, d_bz, FP8_E4,
                    format_delta(FP8_E4, conv));
}

fp8_status_t fp8_linear_dgrad_q(fp8_ctx *ctx, const uint8_t *dy8, const int32_t *d_bg, const uint8_t *w8,
                                const uint8_t *w8_t, const int32_t *d_bw, fp8_act_t act, const void *y_pre, void *dx,
                                void *g, uint8_t *g8, const int32_t *d_bq, float *d_amax_g, int64_t T, int64_t K,
                                int64_t N, fp8_conv_t conv, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !dy8 || !d_bg || (!w8 && !w8_t) || !d_bw || !g8 || !d_bq) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)act < (int)FP8_ACT_NONE || (int)act > (int)FP8_ACT_SWIGLU)
        return FP8_ERR_DTYPE;
    if (act != FP8_ACT_NONE && !y_pre) return FP8_ERR_NULL;
    if (act == FP8_ACT_NONE && (y_pre || dx)) return FP8_ERR_UNSUPPORTED;  // g is the input gradient itself
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    const bool w_mn = (w8_t == nullptr);
    const uint8_t *w = w_mn ? w8 : w8_t;
    if (!aligned16(dy8) || !aligned16(w) || (N % 16) != 0 || (K % (act == FP8_ACT_SWIGLU ? 32 : 16)) != 0 ||
        (y_pre && !aligned16(y_pre)) || !aligned16(g8) || (g && !aligned16(g)) || (dx && !aligned16(dx)))
        return FP8_ERR_ALIGN;
    int delta = format_delta(FP8_E5, conv) + format_delta(FP8_E4, conv);
    const int kind = act == FP8_ACT_GELU ? 2 : (act == FP8_ACT_SWIGLU ? 5 : 3);
    return run_gemm(ctx, dy8, FP8_E5, false, d_bg, w, FP8_E4, w_mn, d_bw, delta, nullptr, 0, dx, FP8_BF16, d_amax_g, T, K,
                    N, (cudaStream_t)stream, kind, g, y_pre, g8, d_bq, FP8_E5, format_delta(FP8_E5, conv));
}

fp8_status_t fp8_linear_f16acc(fp8_ctx *ctx, fp8_matmul_t kind, const uint8_t *a8, const int32_t *d_ba, const uint8_t *b8,
                               const int32_t *d_bb, void *out, fp8_dtype_t out_dt, int32_t chunk, int64_t T, int64_t K,
                               int64_t N, fp8_conv_t conv, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !a8 || !d_ba || !b8 || !d_bb || !out) return FP8_ERR_NULL;
    if ((int)kind < 0 || (int)kind > 2 || (int)conv < 0 || (int)conv > 1 || (int)out_dt < 0 || (int)out_dt > 2) return FP8_ERR_DTYPE;
    if (out_dt != FP8_F16 && out_dt != FP8_F32) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0 || chunk <= 0 || (chunk % kBK) != 0) return FP8_ERR_SHAPE;
    // operands in their forward layouts: X8[T,K], W8[N,K], dY8[T,N]
    const int64_t rows = kind == FP8_MM_WGRAD ? N : T, cols = kind == FP8_MM_FWD ? N : K;
    const int64_t contraction = kind == FP8_MM_FWD ? K : (kind == FP8_MM_DGRAD ? N : T);
    if (!aligned16(a8) || !aligned16(b8) || !aligned16(out) || (K % 16) != 0 || (N % 16) != 0 || (cols % 8) != 0) return FP8_ERR_ALIGN;
    const int e4 = format_delta(FP8_E4, conv), e5 = format_delta(FP8_E5, conv);
    const int a_fmt = kind == FP8_MM_FWD ? FP8_E4 : FP8_E5;
    const int delta = (kind == FP8_MM_FWD ? e4 : e5) + e4;
    const bool a_mn = kind == FP8_MM_WGRAD, b_mn = kind != FP8_MM_FWD;
    return run_gemm(ctx, a8, a_fmt, a_mn, d_ba, b8, FP8_E4, b_mn, d_bb, delta, nullptr, 0, out, (int)out_dt, nullptr, rows, cols,
                    contraction, (cudaStream_t)stream, 6, nullptr, nullptr, nullptr, nullptr, 0, 0, false, chunk / kBK);
}

static fp8_status_t linear_wgrad_impl(fp8_ctx *ctx, const uint8_t *dy8, const uint8_t *dy8_t, const int32_t *d_bg,
                                      const uint8_t *x8, const uint8_t *x8_t, const int32_t *d_bx, void *dw,
                                      fp8_dtype_t dw_dt, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream,
                                      fp8lin::GroupSlot *slot)
{
    using namespace fp8lin;
    if (!ctx || (!dy8 && !dy8_t) || !d_bg || (!x8 && !x8_t) || !d_bx || !dw) return FP8_ERR_NULL;
    if ((int)conv < 0 || (int)conv > 1 || (int)dw_dt < 0 || (int)dw_dt > 2) return FP8_ERR_DTYPE;
    if (!out_dtype_ok(dw_dt)) return FP8_ERR_UNSUPPORTED;
    if (T <= 0 || K <= 0 || N <= 0) return FP8_ERR_SHAPE;
    // each operand comes either as its transposed copy (contraction over contiguous bytes) or as the forward
    // layout dY8[T,N] / X8[T,K] (contraction strided)
    const bool g_mn = (dy8_t == nullptr), x_mn = (x8_t == nullptr);
    const uint8_t *g = g_mn ? dy8 : dy8_t, *xx = x_mn ? x8 : x8_t;
    if (!aligned16(g) || !aligned16(xx) || (!g_mn && (T % 16) != 0) || (!x_mn && (T % 16) != 0) ||
        (g_mn && (N % 16) != 0) || (x_mn && (K % 16) != 0) || (reinterpret_cast<uintptr_t>(dw) & 3u))
        return FP8_ERR_ALIGN;
    int delta = format_delta(FP8_E5, conv) + format_delta(FP8_E4, conv);
    return run_gemm(ctx, g, FP8_E5, g_mn, d_bg, xx, FP8_E4, x_mn, d_bx, delta, nullptr, 0, dw, dw_dt, nullptr, N, K, T,
                    (cudaStream_t)stream, 0, nullptr, nullptr, nullptr, nullptr, 0, 0, false, 0, false, nullptr, slot);
}

fp8_status_t fp8_linear_wgrad(fp8_ctx *ctx, const uint8_t *dy8, const uint8_t *dy8_t, const int32_t *d_bg,
                              const uint8_t *x8, const uint8_t *x8_t, const int32_t *d_bx, void *dw,
                              fp8_dtype_t dw_dt, int64_t T, int64_t K, int64_t N, fp8_conv_t conv, void *stream)
{
    return linear_wgrad_impl(ctx, dy8, dy8_t, d_bg, x8, x8_t, d_bx, dw, dw_dt, T, K, N, conv, stream, nullptr);
}

// One matmul of a group, through the same checks and set-up as its own entry point.
static fp8_status_t group_item_call(fp8_ctx *ctx, const fp8_matmul_item_t &m, fp8_conv_t conv, void *stream,
                                    fp8lin::GroupSlot *slot)
{
    switch (m.kind) {
    case FP8_MATMUL_FWD:
        return linear_fwd_impl(ctx, m.a8, m.d_ba, m.b8, m.d_bb, m.bias_vec, (fp8_dtype_t)m.bias_dt, m.out,
                               (fp8_dtype_t)m.out_dt, m.d_amax_out, m.T, m.K, m.N, conv, stream, slot);
    case FP8_MATMUL_DGRAD:
        return linear_dgrad_impl(ctx, m.a8, m.d_ba, m.b8, nullptr, m.d_bb, m.out, (fp8_dtype_t)m.out_dt, m.d_amax_out, m.T,
                                 m.K, m.N, conv, stream, slot);
    case FP8_MATMUL_WGRAD:
        if (m.d_amax_out) return FP8_ERR_UNSUPPORTED;
        return linear_wgrad_impl(ctx, m.a8, nullptr, m.d_ba, m.b8, nullptr, m.d_bb, m.out, (fp8_dtype_t)m.out_dt, m.T, m.K,
                                 m.N, conv, stream, slot);
    default: return FP8_ERR_DTYPE;
    }
}

fp8_status_t fp8_linear_group(fp8_ctx *ctx, const fp8_matmul_item_t *items, int32_t count, fp8_conv_t conv, void *stream)
{
    using namespace fp8lin;
    if (!ctx || !items) return FP8_ERR_NULL;
    if (count <= 0) return FP8_ERR_SHAPE;
    if ((int)conv < 0 || (int)conv > 1) return FP8_ERR_DTYPE;
    // rows, columns and contraction length of each item as a matmul
    auto dims = [](const fp8_matmul_item_t &m, int64_t &M, int64_t &N, int64_t &Kc) {
        if (m.kind == FP8_MATMUL_FWD) { M = m.T; N = m.N; Kc = m.K; }
        else if (m.kind == FP8_MATMUL_DGRAD) { M = m.T; N = m.K; Kc = m.N; }
        else { M = m.N; N = m.K; Kc = m.T; }
    };
    bool one_launch = count <= kGroupGemmMax && g_max_pairs > 0 && !g_force_single && !g_no_group_gemm;
    bool wide = kWideTileDefault && g_force_wide != 0;
    for (int i = 0; i < count; ++i) {
        if (items[i].kind < 0 || items[i].kind > 2) return FP8_ERR_DTYPE;
        if (items[i].T <= 0 || items[i].K <= 0 || items[i].N <= 0) return FP8_ERR_SHAPE;
        int64_t M, N, Kc;
        dims(items[i], M, N, Kc);
        if (M <= kBM) one_launch = false;   // a decode-size member: its own kernel, its own launch
        if (Kc < 2048 || ((N + 511) / 512) * 512 - N > N / 32) wide = false;   // the wide tile would waste its width
    }
    if (g_force_wide == 1) wide = true;
    if (!one_launch) {
        for (int i = 0; i < count; ++i) {
            const fp8_status_t st = group_item_call(ctx, items[i], conv, stream, nullptr);
            if (st != FP8_OK) return st;
        }
        return FP8_OK;
    }
    // Shortest contractions first.  Where one problem ends and the next begins some pairs are a tile ahead of the
    // others, by the difference of the two tile times, and stay so; pairs that share operand strips hit in L2 only while
    // they walk them at about the same time.  In this order the large differences come last (measured on the twelve
    // matmuls of a 7B-class step: 3.22 ms and 3.3 GB read from DRAM, against 3.27 ms and 4.6 GB longest first, 3.29 ms
    // in the caller's order, 3.38 ms as twelve launches).
    int order[kGroupGemmMax];
    for (int i = 0; i < count; ++i) order[i] = i;
    for (int i = 1; i < count; ++i) {   // insertion sort, stable
        int64_t Mi, Ni, Ki;
        const int oi = order[i];
        dims(items[oi], Mi, Ni, Ki);
        int j = i;
        for (; j > 0; --j) {
            int64_t Mj, Nj, Kj;
            dims(items[order[j - 1]], Mj, Nj, Kj);
            if (g_group_order == 2 || (g_group_order == 1 ? Kj >= Ki : Kj <= Ki)) break;
            order[j] = order[j - 1];
        }
        order[j] = oi;
    }
    static thread_local GroupGemmParams gg;   // about 11 KB: filled per call, copied by the launch
    gg.count = count;
    gg.first_tile[0] = 0;
    for (int i = 0; i < count; ++i) {
        GroupSlot slot = {&gg, i, wide};
        const fp8_status_t st = group_item_call(ctx, items[order[i]], conv, stream, &slot);
        if (st != FP8_OK) return st;   // argument errors surface before anything of the group is launched
        const int64_t tiles = (int64_t)gg.p[i].tiles_m * gg.p[i].tiles_n + gg.first_tile[i];
        if (tiles > 0x7FFFFFFF) return FP8_ERR_SHAPE;
        gg.first_tile[i + 1] = (int)tiles;
    }
    const int total = gg.first_tile[count];
    const int pairs = total < g_max_pairs ? total : g_max_pairs;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * (unsigned)pairs);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = wide ? PairSmemWide::kDynamic : PairSmem::kDynamic;
    cfg.stream = (cudaStream_t)stream;
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    const cudaError_t le = wide ? cudaLaunchKernelEx(&cfg, gemm_pair_group_kernel<2>, gg)
                                : cudaLaunchKernelEx(&cfg, gemm_pair_group_kernel<1>, gg);
    if (le != cudaSuccess) {
        // the launch was refused (the 11 KB of kernel parameters need a driver that takes more than 4 KB): nothing
        // has run, the members go out one by one
        (void)cudaGetLastError();
        for (int i = 0; i < count; ++i) {
            const fp8_status_t st = group_item_call(ctx, items[i], conv, stream, nullptr);
            if (st != FP8_OK) return st;
        }
        return FP8_OK;
    }
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

}  // extern "C"
