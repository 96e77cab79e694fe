// Tensor-core convolution kernels for sm_100a: implicit GEMM on tcgen05.mma (kind::tf32, fp32
// accumulators in tensor memory), operands staged in shared memory by TMA, one elected thread
// issuing the MMAs, mbarrier hand-shakes between the TMA producer, the MMA issuer and the epilogue.
//
// Forward (and the data gradient, which is a forward convolution over dy with rearranged weights):
//   D[pixels, c_out] = sum over taps (r,s) and channel chunks of A_tap[pixels, c] * W_tap[c_out, c]^T
//   One CTA owns one tile of 128 output pixels, chosen as a rectangular box (w x h x n) of the
//   output so that the A operand of every tap is ONE tiled TMA box of the input tensor, shifted by
//   (r - pad, s - pad); TMA's out-of-bounds zero fill is the convolution's zero padding.  Both
//   operands are K-major (channels innermost) with the 64-byte or 128-byte shared-memory swizzle.
//   A strided 1x1 convolution reads its input through a tensor map with doubled strides.
// Weight gradient:
//   dW[c_out, tap, c_in] = sum over pixels dy[pixel, c_out] * x[pixel + tap, c_in]
//   The reduction runs over pixels, but the tensors are channels-innermost, and kind::tf32 reads
//   MN-major shared-memory operands as zeros on this hardware (measured), so both operands must be
//   re-laid K-major (pixels innermost).  TMA brings the raw [pixel][channel] tiles in, four warps
//   transpose them in shared memory into the 128-byte-swizzled K-major layout (4 conflict-free
//   32-bit loads and one 128-bit store per thread and 4 pixels), and the MMA issuer consumes those.
//   One CTA walks a slice of the pixel tiles, keeps one accumulator per tap in tensor memory, and
//   writes a partial; a second kernel adds the partials in fixed order.
//
// Precision.  One TF32 pass keeps 11 significand bits of each operand; through a thousand layers that error
// grows past the parity tolerance (measured: 3e-2 relative at depth 1001).  The default is therefore the
// error-compensated three-pass form: every operand is split x = hi + lo with hi = x with its low 13 significand
// bits cleared (exactly representable in TF32) and lo = x - hi, and the product is accumulated as
// hi*hi + lo*hi + hi*lo in the fp32 accumulator (the dropped lo*lo term is below 2^-22).  Weights are split once
// per step by a preparation kernel; activation tiles are split in shared memory by four warps between the TMA
// arrival and the MMA (the weight gradient's transposing warps do it in the same pass).  The paths are
// HBM/latency bound, so the extra tensor work is hidden.  A one-pass mode remains selectable.
//
// Every wait on an mbarrier is bounded: after the limit the kernel records where it gave up in the
// device status word, stops issuing work, waits (bounded) for its TMA copies in flight, frees its
// tensor memory and returns.
#include "conv_tc.h"

#include <cuda.h>
#include <stdint.h>
#include <string.h>

namespace hpf {

namespace {

constexpr int kTileM = 128;                 // MMA M (TMEM lanes)
constexpr long long kWaitLimit = 4000000000LL;   // clock64 ticks (~2 s) before a wait gives up
constexpr uint32_t kSmemBudget = 200 * 1024;
constexpr uint32_t kWgradSmemBudget = 220 * 1024;   // the weight-gradient kernel has next to no static shared memory
constexpr int kFwdMaxStages = 4;
#ifndef HPF_WGRAD_WANT
#define HPF_WGRAD_WANT 96
#endif
constexpr int kWgradWantCtas = HPF_WGRAD_WANT;   // CTAs a weight-gradient launch spreads its pixel walk over at least
constexpr int kMultiTileFrom = 2 * 296;     // CTAs (two per SM) beyond which a forward / data-gradient launch gives each CTA two tiles
constexpr unsigned int kCellTmemCols = 256;  // tensor-memory columns a persistent cell CTA may hold (two such CTAs share an SM's 512)
constexpr unsigned int kCellSmemBudget = 100 * 1024;   // dynamic shared memory of a cell CTA (two per SM)
constexpr unsigned int kWgradSlack = 16384;   // an MMA reads 128 operand rows (16 KB) from a base that may be the last one in use

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_inval(uint32_t bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait.  Returns false if it gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitLimit) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp receives lane (base lane + i)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// The same without the wait, so that several loads can be in flight before one tmem_ld_wait().
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, float* v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tmap(const void* tmap)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets in
// 16-byte units, descriptor version 1, swizzle mode in the top bits (2 = 128 B, 4 = 64 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle_bytes)
{
    const uint64_t layout = swizzle_bytes == 128 ? 2ull : 4ull;
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (layout << 61);
}

// MN-major TF32 operand (the reduction index runs over the rows of the tile, channels are contiguous): the one layout
// the tensor core accepts for 32-bit MN-major operands is rows of 128 bytes whose 32-byte chunks are XOR-swizzled by
// (row % 4) (layout type 1, what a TMA box with CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B delivers).  One MMA of K = 8 reads
// 8 consecutive rows (two groups of 4, `stride` = 512 bytes apart) of every 32-channel block; `block_bytes` is the
// distance between consecutive 32-channel blocks (the leading-dimension offset).
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t block_bytes)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((block_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((512u >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (1ull << 61);
}

// Instruction descriptor: fp32 accumulator, TF32 A and B, M = 128, N = n; major bits select MN-major operands.
inline uint32_t instr_desc(int n, bool a_mn_major, bool b_mn_major)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

// Optional timelines for latency studies (debug builds only).  HPF_TC_TIMELINE=2: every CTA of the forward kernel
// stamps its milestones in shared memory and adds the elapsed times to per-class totals (class = window size and
// grid size), read back with hpf_debug_timeline.  Otherwise: globaltimer stamps of CTA (0,0) behind the status word.
#if defined(HPF_TC_TIMELINE) && HPF_TC_TIMELINE == 2
__device__ unsigned long long g_tl_acc[8][16];
#define HPF_TL(slot)                                                                                      \
    do {                                                                                                  \
        unsigned long long t_;                                                                            \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                            \
        tl_s[(slot)] = t_;                                                                                \
    } while (0)
#elif defined(HPF_TC_TIMELINE)
#define HPF_TL(slot)                                                                                      \
    do {                                                                                                  \
        if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {                                      \
            unsigned long long t_;                                                                        \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                        \
            reinterpret_cast<unsigned long long*>(p.status)[2 + (slot)] = t_;                             \
        }                                                                                                 \
    } while (0)
#else
#define HPF_TL(slot) do {} while (0)
#endif

__device__ __forceinline__ void report(DeviceStatus* status, unsigned int code)
{
    if (atomicCAS(&status->code, 0u, code) == 0u) status->detail = blockIdx.x;
}

// ------------------------------------------------------------------------------------------------
// kernel parameters
// ------------------------------------------------------------------------------------------------
// The scalar part of the parameters is copied to shared memory by the first warps at kernel start: a kernel
// parameter block of this size spans several constant-cache lines, and first touches from the single-thread
// roles (producer, MMA issuer) and from the epilogue would each pay a serialised miss on the critical path.
struct FwdScalars {
    float* out;
    const float* extra;
    DeviceStatus* status;
    long long os_n, os_h, os_w;  // output strides (floats) of pixel (n, p, q)
    long long dense_h, dense_w;  // strides of one row / one pixel of the dense output (zero fill)
    int accumulate;
    int box_w, box_h, box_n, tiles_w, tiles_h;
    int P, Q, N;                 // output pixel grid of the GEMM
    int c_out, n_chunk;          // total output channels, channels per CTA
    int R, pad;                  // window and the tap shift
    int c_in, kchunk, n_kchunks;
    int swizzle;
    int stages;
    int passes;                  // 1 or 3
    int stacked;                 // three-pass: hi*hi and hi*lo come from one MMA over [B_hi; B_lo] (needs 2*n_chunk <= 256)
    int zero_fill;               // > 1: the output pixel grid is strided, fill the rest of each patch with zeros
    int out_h, out_w;            // dense output extent (zero fill bounds)
    unsigned int a_bytes, b_bytes, stage_bytes, tx_bytes, tmem_cols, idesc, idesc2, stg_pitch;
    // batch-norm statistics folded into the write-out (see ConvBnFuse): 0 none, 1 sums of the output and its square
    int stat_mode;
    float* stat_partials;        // [tiles][2][c_out] per-tile partial sums
    unsigned int* stat_ticket;   // counts finished CTAs; zero between launches
    float* stat_out;             // mean[c_out], rstd[c_out], written by the CTA that finishes last
    float stat_eps;
    float stat_inv_tile_rows;    // 1 / (pixels of one tile)
    double stat_inv_rows;        // 1 / (pixels the statistics run over)
    // BN+ReLU applied to the activation operand on its way to the tensor core (see ConvBnFuse::in_mode)
    // several tiles per CTA (MULTI kernel; tile j of CTA b is tile b*tiles_per_cta + j): tile j+1's loads, split and MMAs
    // run under tile j's write-out, each tile has its own accumulator columns, and the write-out is staged in a region
    // of its own
    int n_tiles, tiles_per_cta;
    unsigned int acc_cols;       // tensor-memory columns of one tile's accumulator
    unsigned int stg_off;        // byte offset of the write-out staging area (0: it reuses the idle pipeline buffers)
    int bn_in;
    int in_w, in_h;              // extent of the input pixel grid (the padding mask)
    const float* bn_in_gamma;
    const float* bn_in_beta;
    const float* bn_in_stats;    // bn_in 1: mean[c_in], rstd[c_in] (left by the kernel that produced x)
    // bn_in 2: the statistics are derived here from the producer's per-tile sums and stored by the first CTA
    const float* bn_in_partials; // [bn_in_tiles][2][c_in]
    float* bn_in_stats_out;
    int bn_in_tiles;
    float bn_in_eps;
    double bn_in_inv_rows;
    float* bn_in_y;              // relu(bn(x)), dense [N][in_h][in_w][c_in], written by the CTAs of the first channel slice
    // K loop split over gridDim.z CTAs (launches of a few tiles with a long K loop): every CTA stores its partial tile, the
    // one that takes the last ticket of its (tile, channel slice) adds them in split order and writes the output
    int pdl_late;                // see the kernel's first statement
    int ksplit;
    float* splitk_partials;      // [(tile * slices + slice) * ksplit + z][128][n_chunk]
    unsigned int* splitk_ticket; // one per (tile, slice); zero between launches
};
struct alignas(64) FwdParams {
    CUtensorMap tm_a;            // activations {C, Wv, Hv, N}
    CUtensorMap tm_b;            // weights, hi part {taps*C, c_out}
    CUtensorMap tm_b_lo;         // weights, lo part (three-pass mode)
    FwdScalars s;
};

struct WgradScalars {
    float* out;                  // dw or partials [splits][c_out*taps*c_in]
    DeviceStatus* status;
    int box_w, box_h, box_n, tiles_w, tiles_h, n_tiles, tiles_per_split;
    int rows;                    // pixel rows of a tile in shared memory (32 or 64)
    int box_rows;                // pixels the copy delivers (<= rows); the rest stays zero
    int c_out, c_in, R, pad;
    int m_chunk;                 // output channels per CTA (<= 128)
    int n_cols;                  // input channels per CTA (<= 256)
    int taps_per_cta;
    int taps_per_mma;            // taps stacked along N in one MMA (n_cols * taps_per_mma <= 256)
    int raw_stages, t_stages;
    int passes;                  // 1 or 3
    unsigned int raw_bytes, t_bytes, tx_per_tap, tx_a, tmem_cols, idesc, idesc_tail;
    long long split_stride;      // floats between partials
};
struct alignas(64) WgradParams {
    CUtensorMap tm_a;            // dy {c_out, Q, P, N}, box {m_chunk, w, h, n}, no swizzle
    CUtensorMap tm_b;            // x {C, Wv, Hv, N}, box {n_cols, w, h, n}, no swizzle
    WgradScalars s;
};

struct WgradDirectScalars {
    float* out;                  // dw or partials [splits][c_out*taps*c_in]
    DeviceStatus* status;
    int box_w, box_h, box_n, tiles_w, tiles_h, n_tiles, tiles_per_split;
    int rows;                    // pixel rows of a tile in shared memory (a multiple of 8)
    int box_rows;                // pixels the copy delivers (<= rows); the rest stays zero
    int c_out, c_in, R, pad;
    int m_chunk, n_cols;         // output / input channels per CTA
    int m_blocks, n_blocks;      // 32-channel blocks of the dy tile / of one tap's x tile (a 16-channel tensor fills half a block)
    int m_box, n_box;            // channels per TMA box: 32, or 16 for a 16-channel tensor
    int taps_per_cta, taps_per_mma;
    int stages, passes;
    unsigned int stage_bytes, lo_off, tx_bytes_a, tx_per_tap, tmem_cols, idesc, idesc_tail;
    long long split_stride;      // floats between partials
};
struct alignas(64) WgradDirectParams {
    CUtensorMap tm_a;            // dy {c_out, Q, P, N}, box {m_box, w, h, n}, 128-byte swizzle with 32-byte atoms
    CUtensorMap tm_b;            // x {C, Wv, Hv, N}, box {n_box, w, h, n}, same swizzle
    WgradDirectScalars s;
};

template <class T>
__device__ __forceinline__ void load_scalars(T* dst, const T* src)
{
    static_assert(sizeof(T) % 4 == 0, "scalar block must be a whole number of words");
    const uint32_t* w = reinterpret_cast<const uint32_t*>(src);
    for (int i = threadIdx.x; i < (int)(sizeof(T) / 4); i += blockDim.x) reinterpret_cast<uint32_t*>(dst)[i] = w[i];
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// x = hi + lo, hi = x with the low 13 significand bits cleared (what a TF32 operand keeps)
__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }

// BN statistics from per-tile moments [n_tiles][2][C]: per tile and channel the mean of the tile's values and the sum
// of their squared deviations from that mean (M2).  Every tile holds the same number of values (the host fuses only
// launches whose tiles are all full), so the total is
//     mean = average of the tile means,   M2 = sum of the tile M2 + n_tile * sum (tile mean - mean)^2,
// evaluated about tile 0's mean so that no difference of large numbers appears anywhere: the result stays accurate
// however far a channel's mean is from zero compared with its spread.  What is added up are small differences of tile
// means, their squares and the non-negative tile M2, at most a few hundred terms: fp32 sums in a fixed order (every
// caller gets the same bits), the final combination in fp64.  Called by 256 threads (tid 0..255) that share named
// barrier 1; C is a power of two in 16..256; bn_ws: 8 x 32 x 8 floats of shared memory.  On return thread tid < C holds
// its channel's mean and 1/sqrt(var + eps).
// Consecutive threads read consecutive float4 of a tile's row (coalesced: every CTA of a launch reads these same few
// lines); the lanes of a warp that share a column are added by a butterfly, the warps through shared memory.
__device__ __forceinline__ void bn_combine_partials(const float* partials, int n_tiles, int C, double inv_rows, float eps,
                                                    float (*bn_ws)[32][8], int tid, float* mean, float* rstd)
{
    const int ncol4 = C >> 1;                          // float4 columns of one tile's [2][C] moments: 8..128
    const int col4 = tid % ncol4, ln = tid / ncol4, L = 256 / ncol4;
    const float4* part = reinterpret_cast<const float4*>(partials);
    // the first C/4 columns are tile means: accumulated as differences from tile 0's mean (and their squares)
    const bool mean_col = col4 < (C >> 2);
    const float4 ref = mean_col ? __ldcg(part + col4) : make_float4(0.f, 0.f, 0.f, 0.f);
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f, b0 = 0.f, b1 = 0.f, b2 = 0.f, b3 = 0.f;
    // eight rows per batch, all eight loads in flight together (a loop that used each load before issuing the next would
    // pay an L2 round trip per row); rows beyond the last add zero
    for (int k0 = ln; k0 < n_tiles; k0 += 8 * L) {
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = k0 + j * L;
            v[j] = k < n_tiles ? __ldcg(part + (size_t)k * ncol4 + col4) : ref;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float f0 = v[j].x - ref.x, f1 = v[j].y - ref.y, f2 = v[j].z - ref.z, f3 = v[j].w - ref.w;
            a0 += f0; a1 += f1; a2 += f2; a3 += f3;
            b0 = fmaf(f0, f0, b0); b1 = fmaf(f1, f1, b1); b2 = fmaf(f2, f2, b2); b3 = fmaf(f3, f3, b3);
        }
    }
    // lanes of one warp that share a column (fewer than 32 columns): a fixed butterfly
    for (int off = 16; off >= ncol4; off >>= 1) {
        a0 += __shfl_xor_sync(0xffffffffu, a0, off); a1 += __shfl_xor_sync(0xffffffffu, a1, off);
        a2 += __shfl_xor_sync(0xffffffffu, a2, off); a3 += __shfl_xor_sync(0xffffffffu, a3, off);
        b0 += __shfl_xor_sync(0xffffffffu, b0, off); b1 += __shfl_xor_sync(0xffffffffu, b1, off);
        b2 += __shfl_xor_sync(0xffffffffu, b2, off); b3 += __shfl_xor_sync(0xffffffffu, b3, off);
    }
    const int warp = tid >> 5, lane = tid & 31;
    if (lane < ncol4) {
        float* d = bn_ws[warp][lane];
        *reinterpret_cast<float4*>(d) = make_float4(a0, a1, a2, a3);
        if (mean_col) *reinterpret_cast<float4*>(d + 4) = make_float4(b0, b1, b2, b3);
    }
    // tile 0's means travel in the half of an M2 column's slot that nothing else uses (that of the channel's M2 column in
    // the first warp that holds it), so that nothing has to be fetched again after the barrier
    if (mean_col && ln == 0) {
        const int qv0 = (C >> 2) + col4;
        *reinterpret_cast<float4*>(bn_ws[ncol4 > 32 ? qv0 >> 5 : 0][qv0 & 31] + 4) = ref;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (tid < C) {
        // column q sits in lane q % 32 of the warps q / 32, q / 32 + ncol4 / 32, ... (of every warp when there are at most
        // 32 columns): added in ascending warp order
        const int qm = tid >> 2, qv = (C >> 2) + (tid >> 2), comp = tid & 3;
        const int wstep = ncol4 > 32 ? ncol4 >> 5 : 1;
        float sd = 0.f, sq = 0.f, m2 = 0.f;
        for (int w = (ncol4 > 32 ? qm >> 5 : 0); w < 8; w += wstep) { sd += bn_ws[w][qm & 31][comp]; sq += bn_ws[w][qm & 31][4 + comp]; }
        for (int w = (ncol4 > 32 ? qv >> 5 : 0); w < 8; w += wstep) m2 += bn_ws[w][qv & 31][comp];
        // (no fp64 division: mean = ref + sd / T and var = M2 / rows + (sq - sd^2 / T) / T with 1 / T in fp32-exact steps)
        const double inv_tiles = (double)(1.0f / (float)n_tiles);
        const double dsd = (double)sd;
        const double m = (double)bn_ws[ncol4 > 32 ? qv >> 5 : 0][qv & 31][4 + comp] + dsd * inv_tiles;
        double var = (double)m2 * inv_rows + ((double)sq - dsd * dsd * inv_tiles) * inv_tiles;
        if (var < 0.0) var = 0.0;
        *mean = (float)m;
        *rstd = 1.0f / sqrtf((float)(var + (double)eps));          // correctly rounded fp32 operations: within an ulp or two of the fp64 result
    }
}

// ------------------------------------------------------------------------------------------------
// forward / data-gradient kernel: 10 warps = TMA producer, MMA issuer, 8 splitter / epilogue warps
// ------------------------------------------------------------------------------------------------
// One CTA's share of a forward / data-gradient launch: `vb` of `vg` (block index and grid size of the launch as a stand-alone
// launch has them).  MODE 0: one 128-pixel tile per CTA (the shortest launch; what a launch of up to one wave wants).
// MODE 1: p.tiles_per_cta tiles per CTA for launches of several waves: fewer CTAs, and a tile's write-out hides the next
// tile's loads, split and MMAs.  MODE 2: the K loop split over vg.z CTAs.  MODE 3: inside the persistent cell kernel, which
// runs many launches one after the other in one resident grid: tiles per CTA and K split are read from the parameters,
// tensor memory is allocated once by the caller, the mbarriers are set up again for every call, and nothing of the
// programmatic-launch protocol applies.  `p` (shared memory) holds gp->s.
template <int MODE>
__device__ __forceinline__ int conv_fwd_cta(const FwdParams* gpp, FwdScalars& p, const uint3 vb, const uint3 vg, const uint32_t cell_tmem_base,
                                             const bool cell_first)
{
    const FwdParams& gp = *gpp;
    constexpr bool CELL = MODE == 3;
    const bool MULTI = CELL ? p.tiles_per_cta > 1 : MODE == 1;
    const bool KSPLIT = CELL ? p.ksplit > 1 : MODE == 2;
#if defined(HPF_TC_TIMELINE) && HPF_TC_TIMELINE == 2
    __shared__ unsigned long long tl_s[16];
    if (threadIdx.x < 16) tl_s[threadIdx.x] = 0;
#endif
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[3 * 8 + 4];       // full[8], empty[8], split[8], accum[4] (one per tile of this CTA)
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued, consumed;

    const uint32_t base_off = ((smem_u32(smem_raw) + 1023u) & ~1023u) - smem_u32(smem_raw);
    uint8_t* smem = smem_raw + base_off;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[8]), split0 = smem_u32(&bars[16]),
                   accum_bar = smem_u32(&bars[24]);
    // stage layout: A | A_lo | B_hi | B_lo   (the lo parts only in three-pass mode)
    const uint32_t off_alo = p.a_bytes;
    const uint32_t off_b = p.passes == 3 ? 2 * p.a_bytes : p.a_bytes;
    const uint32_t off_blo = off_b + p.b_bytes;

    const int tiles_per_cta = MULTI ? p.tiles_per_cta : 1;
    const int tile0 = (int)vb.x * tiles_per_cta;
    const int my_tiles = MULTI ? (p.n_tiles - tile0 < tiles_per_cta ? p.n_tiles - tile0 : tiles_per_cta) : 1;
    const uint32_t acc_cols = MULTI ? p.acc_cols : 0u;
    const uint32_t stg_off = MULTI ? p.stg_off : 0u;
    const int co0 = (int)vb.y * p.n_chunk;
    // first pixel (q0, p0, n0) of tile t
#define HPF_TILE_ORIGIN(t_)                                                          \
    int q0, p0, n0;                                                                   \
    {                                                                                 \
        int t__ = (t_);                                                               \
        const int tw__ = t__ % p.tiles_w; t__ /= p.tiles_w;                           \
        q0 = tw__ * p.box_w; p0 = (t__ % p.tiles_h) * p.box_h; n0 = (t__ / p.tiles_h) * p.box_n; \
    }

    if (threadIdx.x == 0) HPF_TL(0);
    const int total = p.R * p.R * p.n_kchunks;
    // this CTA's share of the K loop (all of it unless the launch splits K over gridDim.z)
    const int kb = KSPLIT ? (int)(((long long)total * vb.z) / p.ksplit) : 0;
    const int ke = KSPLIT ? (int)(((long long)total * (vb.z + 1)) / p.ksplit) : total;
    // Thread 0 is the TMA producer.  The origin of its first tile and its first K step are a chain of dependent
    // shared-memory reads and integer divisions in ONE thread (most of a microsecond): worked out here, while the CTA
    // still waits for tensor memory and for the preceding kernel, not between that wait and the first copy.
    int f_q0 = 0, f_p0 = 0, f_n0 = 0, f_tap = 0, f_kc = 0, f_r = 0, f_sx = 0;
    if (threadIdx.x == 0) {
        HPF_TILE_ORIGIN(tile0);
        f_q0 = q0; f_p0 = p0; f_n0 = n0;
        if (KSPLIT) { f_tap = kb / p.n_kchunks; f_kc = kb % p.n_kchunks; f_r = f_tap / p.R; f_sx = f_tap % p.R; }
    }
    if (threadIdx.x == 0) {
        if (CELL && !cell_first)       // the barriers of the call before are retired first
            for (int j = 0; j < 3 * 8 + 4; ++j) mbar_inval(full0 + 8 * j);
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); mbar_init(split0 + 8 * s, 8); }
        for (int j = 0; j < 4; ++j) mbar_init(accum_bar + 8 * j, 1);
        abort_flag = 0; issued = 0; consumed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x == 32) { prefetch_tmap(&gp.tm_a); prefetch_tmap(&gp.tm_b); if (p.passes == 3) prefetch_tmap(&gp.tm_b_lo); }
    if (!CELL && warp == 0) tmem_alloc(smem_u32(&tmem_slot), p.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Everything above touched only parameters, shared and tensor memory.  The TMA producer (thread 0) first works out
    // its first tile's coordinates - a chain of dependent shared-memory reads and integer divisions of most of a
    // microsecond - and waits for the preceding kernel only then, right before its first copy.
    if (!CELL && threadIdx.x != 0) pdl_wait();
    const uint32_t tmem_base = CELL ? cell_tmem_base : tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            // no division in the loop: stage, parity, tap and K chunk are counters
            int it = 0, st = 0;
            uint32_t par = 1u;
            bool live = true;
            const int stages = p.stages, nkc = p.n_kchunks, R = p.R, pad = p.pad, kchunk = p.kchunk, c_in = p.c_in;
            const uint32_t tx = p.tx_bytes, stage_bytes = p.stage_bytes;
            const bool three = p.passes == 3;
            for (int j = 0; j < my_tiles && live; ++j) {
                int q0 = f_q0, p0 = f_p0, n0 = f_n0;
                if (j > 0) {
                    int t__ = tile0 + j;
                    const int tw__ = t__ % p.tiles_w; t__ /= p.tiles_w;
                    q0 = tw__ * p.box_w; p0 = (t__ % p.tiles_h) * p.box_h; n0 = (t__ / p.tiles_h) * p.box_n;
                }
                int tap = f_tap, kc = f_kc, r = f_r, sx = f_sx;
                for (int k = kb; k < ke; ++k, ++it) {
                    if (!mbar_wait(empty0 + 8 * st, par, &abort_flag)) { report(p.status, 1); live = false; break; }
                    const uint32_t dst = smem_base + st * stage_bytes;
                    const int cx = kc * kchunk, cq = q0 + sx - pad, cp = p0 + r - pad, cb = tap * c_in + cx;
                    if (!CELL && it == 0) { pdl_wait(); HPF_TL(1); }
                    mbar_expect_tx(full0 + 8 * st, tx);
                    tma_load_4d(dst, &gp.tm_a, full0 + 8 * st, cx, cq, cp, n0);
                    tma_load_2d(dst + off_b, &gp.tm_b, full0 + 8 * st, cb, co0);
                    if (three) tma_load_2d(dst + off_blo, &gp.tm_b_lo, full0 + 8 * st, cb, co0);
                    if (it == 0) HPF_TL(2);
                    if (++kc == nkc) { kc = 0; ++tap; if (++sx == R) { sx = 0; ++r; } }
                    if (++st == stages) { st = 0; par ^= 1u; }
                }
            }
            if (!CELL && it == 0) pdl_wait();         // nothing to copy: still ordered behind the preceding kernel
            if (CELL && live) {
                // The MMA issuer's last commits on the `empty` barriers are awaited by nobody in a stand-alone launch.  Here
                // the barriers are set up again for the next call, so every arrival still on its way has to land first.
                const int left = it < stages ? it : stages;
                for (int j = 0; j < left; ++j) {
                    if (!mbar_wait(empty0 + 8 * st, par, &abort_flag)) { report(p.status, 8); break; }
                    if (++st == stages) { st = 0; par ^= 1u; }
                }
            }
            issued = it;
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            // One thread issues every MMA, so the loop is kept to a few instructions per MMA: the descriptor's
            // constant part is built once and only its 14-bit address field is advanced (32 bytes = 2 units per K step).
            const uint32_t sbo = 8u * (uint32_t)p.kchunk * 4u;          // 8 rows of one swizzle atom
            const uint64_t desc_hi = smem_desc(0, 16, sbo, p.swizzle);
            const uint32_t idesc = p.idesc, idesc2 = p.idesc2, stage_bytes = p.stage_bytes;
            const bool stacked = p.stacked != 0;
            const int stages = p.stages, k8n = p.kchunk / 8;
            const bool three = p.passes == 3;
            // the splitter warps write the lo part (and with BN+ReLU on the way in rewrite the tile) before the MMAs of the
            // stage are issued.  (Issuing the MMAs that read only the tile as copied ahead of the splitters' barrier was
            // measured: the step got 1.7 ms slower.)
            const bool split_first = three || p.bn_in != 0;
            int it = 0, s = 0;
            uint32_t par = 0;
            bool live = true;
            for (int j = 0; j < my_tiles && live; ++j) {
              const uint32_t acc = tmem_base + (uint32_t)j * acc_cols;
              for (int k = kb; k < ke; ++k, ++it) {
                if (!mbar_wait(full0 + 8 * s, par, &abort_flag)) { report(p.status, 2); live = false; break; }
                if (split_first && !mbar_wait(split0 + 8 * s, par, &abort_flag)) { report(p.status, 6); live = false; break; }
                tc_fence_after();
                if (it == 0) HPF_TL(5);
                const uint32_t st = smem_base + s * stage_bytes;
                const uint64_t a0 = desc_hi | (uint64_t)((st & 0x3FFFFu) >> 4);
                const uint64_t b0 = desc_hi | (uint64_t)(((st + off_b) & 0x3FFFFu) >> 4);
                const uint64_t al0 = desc_hi | (uint64_t)(((st + off_alo) & 0x3FFFFu) >> 4);
                const uint64_t bl0 = desc_hi | (uint64_t)(((st + off_blo) & 0x3FFFFu) >> 4);
                if (three && stacked) {
                    // B_lo follows B_hi in shared memory: A_hi x [B_hi; B_lo] in one MMA of twice the width
                    // (columns [0,n) = hi*hi, [n,2n) = hi*lo, added in the epilogue), then A_lo x B_hi.
#pragma unroll 4
                    for (int k8 = 0; k8 < k8n; ++k8) {
                        umma_tf32(acc, a0 + 2 * k8, b0 + 2 * k8, idesc2, ((k - kb) | k8) ? 1u : 0u);
                        umma_tf32(acc, al0 + 2 * k8, b0 + 2 * k8, idesc, 1u);
                    }
                } else if (three) {
#pragma unroll 4
                    for (int k8 = 0; k8 < k8n; ++k8) {
                        umma_tf32(acc, a0 + 2 * k8, b0 + 2 * k8, idesc, ((k - kb) | k8) ? 1u : 0u);
                        umma_tf32(acc, al0 + 2 * k8, b0 + 2 * k8, idesc, 1u);
                        umma_tf32(acc, a0 + 2 * k8, bl0 + 2 * k8, idesc, 1u);
                    }
                } else {
#pragma unroll 4
                    for (int k8 = 0; k8 < k8n; ++k8) umma_tf32(acc, a0 + 2 * k8, b0 + 2 * k8, idesc, ((k - kb) | k8) ? 1u : 0u);
                }
                umma_commit(empty0 + 8 * s);     // frees the stage once these MMAs have read it
                if (++s == stages) { s = 0; par ^= 1u; }
              }
              if (live) umma_commit(accum_bar + 8 * j);      // tile j's accumulator is complete once these MMAs retire
            }
            consumed = it;
            HPF_TL(6);
        }
    } else {
        // ---- warps 2..9: split the activation tile into hi / lo, then the epilogue ----
        const int tid = threadIdx.x - 64;               // 0..255
        bool ok = true;
        if (p.bn_in) {
            // ---- BN+ReLU on the way in: the tile holds the BN's input x; the operand is relu(gamma*xhat+beta) ----
            __shared__ __align__(16) float bn_par[4][256];      // mean, rstd, gamma, beta per input channel
            const int C = p.c_in;
            if (p.bn_in == 2) {
                // The producer left only its per-tile sums (few enough that adding them here, under the first copy's
                // latency, is cheaper than a ticket at the producer's end): every CTA adds them in the same fixed order,
                // so all CTAs hold identical statistics; the first CTA stores them for the backward pass.
                __shared__ __align__(16) float bn_red[8][32][8];
                float gam = 0.f, bet = 0.f, mu = 0.f, rs = 0.f;
                if (tid < C) { gam = __ldg(p.bn_in_gamma + tid); bet = __ldg(p.bn_in_beta + tid); }   // travel with the sums
                bn_combine_partials(p.bn_in_partials, p.bn_in_tiles, C, p.bn_in_inv_rows, p.bn_in_eps, bn_red, tid, &mu, &rs);
                if (tid < C) {
                    bn_par[0][tid] = mu; bn_par[1][tid] = rs; bn_par[2][tid] = gam; bn_par[3][tid] = bet;
                    if (vb.x == 0 && vb.y == 0) { p.bn_in_stats_out[tid] = mu; p.bn_in_stats_out[C + tid] = rs; }
                }
            }
            // the statistics written by the kernel before (not the read-only path) and the parameters: fetched now, used
            // after the index arithmetic below, which runs under their latency
            float ld_mu = 0.f, ld_rs = 0.f, ld_g = 0.f, ld_b = 0.f;
            if (p.bn_in != 2 && tid < C) {
                ld_mu = __ldcg(p.bn_in_stats + tid); ld_rs = __ldcg(p.bn_in_stats + C + tid);
                ld_g = __ldg(p.bn_in_gamma + tid); ld_b = __ldg(p.bn_in_beta + tid);
            }
            // A thread owns one 16-byte column of the (swizzled) tile rows tid/f4row + j*(256/f4row): its four
            // channels within the K chunk are fixed, and so are the pixels of its rows.
            const int f4row = p.kchunk >> 2;                    // 4 or 8 float4 per tile row
            const int per = (int)(p.a_bytes >> 12);             // rows per thread: 2 or 4
            const int row0 = tid / f4row, rstep = 256 / f4row;
            const int cph = tid % f4row;
            const int clog = p.kchunk == 32 ? (cph ^ (row0 & 7)) : (cph ^ ((row0 >> 1) & 3));
            const bool three = p.passes == 3;
            const bool writer = vb.y == 0;
            const int stages = p.stages, nkc = p.n_kchunks, R = p.R, pad = p.pad;
            // position of row r of the pixel box (the same for every tile)
            int rw[4], rh[4], rn[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = row0 + j * rstep;
                rw[j] = r % p.box_w; rh[j] = (r / p.box_w) % p.box_h; rn[j] = r / (p.box_w * p.box_h);
            }
            const int tap_b = kb / nkc, kc_b = kb - tap_b * nkc, ry_b = tap_b / R, sx_b = tap_b - ry_b * R;
            if (p.bn_in != 2 && tid < C) { bn_par[0][tid] = ld_mu; bn_par[1][tid] = ld_rs; bn_par[2][tid] = ld_g; bn_par[3][tid] = ld_b; }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            int it = 0, s = 0;
            uint32_t par = 0;
            for (int tj = 0; tj < my_tiles && ok; ++tj) {
              HPF_TILE_ORIGIN(tile0 + tj);
              int px[4], py[4], pn[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                px[j] = q0 + rw[j]; py[j] = p0 + rh[j];
                pn[j] = (j < per && rn[j] < p.box_n && n0 + rn[j] < p.N) ? n0 + rn[j] : -1;
              }
              int kc = kc_b, ry = ry_b, sx = sx_b;
              for (int k = kb; k < ke; ++k, ++it) {
                ok = mbar_wait(full0 + 8 * s, par, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) report(p.status, 7); break; }
                if (it == 0 && tid == 0) HPF_TL(3);
                const int dyy = ry - pad, dxx = sx - pad;
                const int ch = kc * p.kchunk + 4 * clog;
                const float4 mu = *reinterpret_cast<const float4*>(&bn_par[0][ch]);
                const float4 rs = *reinterpret_cast<const float4*>(&bn_par[1][ch]);
                const float4 g = *reinterpret_cast<const float4*>(&bn_par[2][ch]);
                const float4 b = *reinterpret_cast<const float4*>(&bn_par[3][ch]);
                float4* a = reinterpret_cast<float4*>(smem + s * p.stage_bytes);
                float4* alo = reinterpret_cast<float4*>(smem + s * p.stage_bytes + off_alo);
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) if (j < per) v[j] = a[tid + 256 * j];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < per) {
                        const int xx = px[j] + dxx, yy = py[j] + dyy;
                        const bool inside = pn[j] >= 0 && (unsigned)xx < (unsigned)p.in_w && (unsigned)yy < (unsigned)p.in_h;
                        float4 y;       // the padding ring is zero AFTER the activation
                        y.x = inside ? fmaxf(fmaf(g.x, (v[j].x - mu.x) * rs.x, b.x), 0.f) : 0.f;
                        y.y = inside ? fmaxf(fmaf(g.y, (v[j].y - mu.y) * rs.y, b.y), 0.f) : 0.f;
                        y.z = inside ? fmaxf(fmaf(g.z, (v[j].z - mu.z) * rs.z, b.z), 0.f) : 0.f;
                        y.w = inside ? fmaxf(fmaf(g.w, (v[j].w - mu.w) * rs.w, b.w), 0.f) : 0.f;
                        if (writer && inside && dxx == 0 && dyy == 0)     // each pixel is some tile's centre tap exactly once
                            *reinterpret_cast<float4*>(p.bn_in_y + (((size_t)pn[j] * p.in_h + yy) * p.in_w + xx) * C + ch) = y;
                        if (three) {
                            const float4 h = make_float4(tf32_hi(y.x), tf32_hi(y.y), tf32_hi(y.z), tf32_hi(y.w));
                            a[tid + 256 * j] = h;
                            alo[tid + 256 * j] = make_float4(y.x - h.x, y.y - h.y, y.z - h.z, y.w - h.w);
                        } else {
                            a[tid + 256 * j] = y;
                        }
                    }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(split0 + 8 * s);
                if (it == 0 && tid == 0) HPF_TL(4);
                if (++kc == nkc) { kc = 0; if (++sx == R) { sx = 0; ++ry; } }
                if (++s == stages) { s = 0; par ^= 1u; }
              }
            }
        } else if (p.passes == 3) {
            const int per = (int)(p.a_bytes >> 12);     // float4 per thread: a_bytes / 16 / 256 = 2 or 4
            const int all = my_tiles * (ke - kb);
            const int stages = p.stages;
            int s = 0;
            uint32_t par = 0;
            for (int it = 0; it < all; ++it) {
                ok = mbar_wait(full0 + 8 * s, par, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) report(p.status, 7); break; }
                if (it == 0 && tid == 0) HPF_TL(3);
                float4* a = reinterpret_cast<float4*>(smem + s * p.stage_bytes);
                float4* alo = reinterpret_cast<float4*>(smem + s * p.stage_bytes + off_alo);
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) if (j < per) v[j] = a[tid + 256 * j];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < per) {
                        // The tile itself stays as copied: the tensor core ignores the 13 low mantissa bits of a 32-bit
                        // operand, which is the very truncation the hi part is defined by.
                        const float4 h = make_float4(tf32_hi(v[j].x), tf32_hi(v[j].y), tf32_hi(v[j].z), tf32_hi(v[j].w));
                        alo[tid + 256 * j] = make_float4(v[j].x - h.x, v[j].y - h.y, v[j].z - h.z, v[j].w - h.w);
                    }
                fence_async_smem();               // generic-proxy writes -> tensor-core reads
                __syncwarp();
                if (lane == 0) mbar_arrive(split0 + 8 * s);
                if (it == 0 && tid == 0) HPF_TL(4);
                if (++s == stages) { s = 0; par ^= 1u; }
            }
        }
        (void)ok;
        // The write-out is staged through shared memory so that it is coalesced (a TMEM lane is a pixel: thread-per-row
        // stores would touch 32 lines each).  With one tile per CTA the staging area is the pipeline itself, idle once
        // the accumulator is complete; with several tiles it is a region of its own, because the next tile's loads and
        // MMAs are in flight while this tile is written out.
        __shared__ float4 shift_s[64];                 // per group of 4 output channels: the shift of the tile's statistics
        __shared__ int row_off[kTileM];                // offset (floats) of the pixel's channel row in the output, or -1
        __shared__ int row_fill[kTileM];               // strided data gradient: which neighbours of the sample exist
        float* const stg = reinterpret_cast<float*>(smem + stg_off);
        bool all_done = true;
        for (int tj = 0; tj < my_tiles; ++tj) {
        HPF_TILE_ORIGIN(tile0 + tj);
        // the row tables do not depend on the accumulator: they are built while the MMAs still run
        if (tid < kTileM) {
            const int wi = tid % p.box_w, hi = (tid / p.box_w) % p.box_h, ni = tid / (p.box_w * p.box_h);
            const int q = q0 + wi, pp = p0 + hi, n = n0 + ni;
            const bool valid = ni < p.box_n && q < p.Q && pp < p.P && n < p.N;
            row_off[tid] = valid ? (int)(n * p.os_n + pp * p.os_h + q * p.os_w + co0) : -1;
            int fill = 0;                              // bit (dy*4 + dx) set: position (pp*s+dy, q*s+dx) gets zeros
            for (int dy = 0; dy < p.zero_fill; ++dy)
                for (int dx = 0; dx < p.zero_fill; ++dx)
                    if ((dy | dx) && pp * p.zero_fill + dy < p.out_h && q * p.zero_fill + dx < p.out_w) fill |= 1 << (dy * 4 + dx);
            row_fill[tid] = (valid && p.zero_fill > 1 && p.zero_fill <= 4) ? fill : 0;
        }
        mbar_wait(accum_bar + 8 * tj, 0, &abort_flag);
        if (!CELL && tj == 0 && p.pdl_late) pdl_launch_dependents();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        const bool done = abort_flag == 0;             // uniform over the 8 warps after the barrier
        all_done = all_done && done;
        if (done) {
            tc_fence_after();
            if (tid == 0 && tj == 0) HPF_TL(7);
            // TMEM lane = pixel within the tile.  Two warps share each group of 32 lanes (a warp reaches lanes
            // 32*(warp%4) ..): they take alternate groups of 16 output channels.
            const int row = (warp & 3) * 32 + lane;
            const int half = (warp - 2) >> 2;
            const uint32_t lane_addr = tmem_base + (uint32_t)tj * acc_cols + ((uint32_t)((warp & 3) * 32) << 16);
            for (int g0 = half * 16; g0 < p.n_chunk; g0 += 32) {
                float v[16];
                tmem_ld16_nowait(lane_addr + (uint32_t)g0, v);
                if (p.stacked) {
                    float u[16];
                    tmem_ld16_nowait(lane_addr + (uint32_t)(p.n_chunk + g0), u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] += u[j];
                } else {
                    tmem_ld_wait();
                }
                float4* dst = reinterpret_cast<float4*>(stg + (size_t)row * p.stg_pitch + g0);
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            }
            if (tid == 0 && tj == 0) HPF_TL(10);
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (tid == 0 && tj == 0) HPF_TL(11);
            bool write_out = true;
            if (KSPLIT) {
                // split K: the staged tile is this CTA's partial sum.  Store it; the CTA that takes the last ticket of this
                // (tile, channel slice) adds all partial tiles in split order (so the sum does not depend on which CTA that
                // is) and goes on to the write-out; the others are done.
                __shared__ int last_of_unit;
                const int c4n_ = p.n_chunk >> 2, tile_f4 = kTileM * c4n_;
                const unsigned int unit = vb.x * vg.y + vb.y;
                float4* mine = reinterpret_cast<float4*>(p.splitk_partials) + ((size_t)unit * p.ksplit + vb.z) * tile_f4;
                for (int idx = tid; idx < tile_f4; idx += 256) {
                    const int r = idx / c4n_, c4 = idx - r * c4n_;
                    mine[idx] = *reinterpret_cast<const float4*>(stg + (size_t)r * p.stg_pitch + 4 * c4);
                }
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (tid == 0) last_of_unit = atomicAdd(p.splitk_ticket + unit, 1u) == (unsigned int)p.ksplit - 1u;
                asm volatile("bar.sync 1, 256;" ::: "memory");
                write_out = last_of_unit != 0;
                if (write_out) {
                    __threadfence();
                    const float4* all = reinterpret_cast<const float4*>(p.splitk_partials) + (size_t)unit * p.ksplit * tile_f4;
                    for (int idx = tid; idx < tile_f4; idx += 256) {
                        float4 a4 = __ldcg(all + idx);
                        for (int z = 1; z < p.ksplit; ++z) {
                            const float4 b4 = __ldcg(all + (size_t)z * tile_f4 + idx);
                            a4.x += b4.x; a4.y += b4.y; a4.z += b4.z; a4.w += b4.w;
                        }
                        const int r = idx / c4n_, c4 = idx - r * c4n_;
                        *reinterpret_cast<float4*>(stg + (size_t)r * p.stg_pitch + 4 * c4) = a4;
                    }
                    if (tid == 0) p.splitk_ticket[unit] = 0u;
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                }
            }
            float4 sa = make_float4(0.f, 0.f, 0.f, 0.f), sb = sa, sk = sa;
            if (write_out) {
            // write-out: consecutive threads write consecutive float4 of a pixel's channel row.  Eight warps cannot
            // hide latency by occupancy, so four independent float4 are in flight per thread and nothing is re-read.
            const int c4n = p.n_chunk >> 2;
            const int total4 = kTileM * c4n;
            const int sh = (c4n & (c4n - 1)) == 0 ? 31 - __clz(c4n) : -1;
            const float* extra = p.extra;
            float* outp = p.out;
            const bool accumulate = p.accumulate != 0;
            const unsigned int pitch = p.stg_pitch;
            const long long dense_h = p.dense_h, dense_w = p.dense_w;
            const int stat_mode = p.stat_mode;
            if (stat_mode) {
                // The statistics are accumulated as deviations from the tile's first pixel (what the kernel stores for it,
                // so residual included): sums of x and x*x themselves would cancel catastrophically in var = E[x^2] - mean^2
                // for a channel whose mean is large compared with its spread.  A thread keeps one group of 4 channels
                // throughout (256 is a multiple of c4n), so one shift per thread does.
                const int c4k = tid % c4n;
                sk = *reinterpret_cast<const float4*>(stg + 4 * c4k);
                if (extra) { const float4 e = __ldcg(reinterpret_cast<const float4*>(extra + row_off[0] + 4 * c4k)); sk.x += e.x; sk.y += e.y; sk.z += e.z; sk.w += e.w; }
                if (accumulate) { const float4 e = *reinterpret_cast<const float4*>(outp + row_off[0] + 4 * c4k); sk.x += e.x; sk.y += e.y; sk.z += e.z; sk.w += e.w; }
                if (tid < c4n) shift_s[tid] = sk;          // read again when the tile's moments are formed
            }
            if (tid == 0 && tj == 0) HPF_TL(12);
            for (int base = tid; base < total4; base += 1024) {
                float4 o[4];
                int off[4];
                int fill[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = base + 256 * u;
                    off[u] = -1; fill[u] = 0;
                    if (idx < total4) {
                        const int r = sh >= 0 ? (idx >> sh) : (idx / c4n);
                        const int c4 = idx - r * c4n;
                        const int ro = row_off[r];
                        if (ro >= 0) {
                            off[u] = ro + 4 * c4;
                            fill[u] = row_fill[r];
                            o[u] = *reinterpret_cast<const float4*>(stg + (size_t)r * pitch + 4 * c4);
                        }
                    }
                }
                if (extra) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (off[u] >= 0) { const float4 e = __ldcg(reinterpret_cast<const float4*>(extra + off[u])); o[u].x += e.x; o[u].y += e.y; o[u].z += e.z; o[u].w += e.w; }
                }
                if (accumulate) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (off[u] >= 0) { const float4 e = *reinterpret_cast<const float4*>(outp + off[u]); o[u].x += e.x; o[u].y += e.y; o[u].z += e.z; o[u].w += e.w; }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (off[u] < 0) continue;
                    float* optr = outp + off[u];
                    *reinterpret_cast<float4*>(optr) = o[u];
                    if (stat_mode) {
                        const float dx_ = o[u].x - sk.x, dy_ = o[u].y - sk.y, dz_ = o[u].z - sk.z, dw_ = o[u].w - sk.w;
                        sa.x += dx_; sa.y += dy_; sa.z += dz_; sa.w += dw_;
                        sb.x = fmaf(dx_, dx_, sb.x); sb.y = fmaf(dy_, dy_, sb.y);
                        sb.z = fmaf(dz_, dz_, sb.z); sb.w = fmaf(dw_, dw_, sb.w);
                    }
                    if (fill[u]) {
                        // strided data gradient: the positions between the samples receive no contribution
                        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int dy = 0; dy < 4; ++dy)
                            for (int dx = 0; dx < 4; ++dx)
                                if (fill[u] & (1 << (dy * 4 + dx))) *reinterpret_cast<float4*>(optr + dy * dense_h + dx * dense_w) = z;
                    }
                }
            }
            }   // write_out
            if (tid == 0 && tj == 0) HPF_TL(13);
            if (p.stat_mode) {
                const int c4n = p.n_chunk >> 2;
                const int stat_mode = p.stat_mode;
                // a thread kept one group of 4 channels throughout (256 is a multiple of c4n): add the 256 / c4n
                // threads of each group in ascending order and store this tile's partial sums
                asm volatile("bar.sync 1, 256;" ::: "memory");          // the staging area is free again
                float4* red = reinterpret_cast<float4*>(stg);
                int n_rows = 256;                                       // rows of `red` per group stride c4n
                if (c4n <= 16) {
                    // the 32 / c4n threads of a group inside a warp first: a fixed butterfly, then one row per warp
                    for (int off = 16; off >= c4n; off >>= 1) {
                        sa.x += __shfl_xor_sync(0xffffffffu, sa.x, off); sa.y += __shfl_xor_sync(0xffffffffu, sa.y, off);
                        sa.z += __shfl_xor_sync(0xffffffffu, sa.z, off); sa.w += __shfl_xor_sync(0xffffffffu, sa.w, off);
                        sb.x += __shfl_xor_sync(0xffffffffu, sb.x, off); sb.y += __shfl_xor_sync(0xffffffffu, sb.y, off);
                        sb.z += __shfl_xor_sync(0xffffffffu, sb.z, off); sb.w += __shfl_xor_sync(0xffffffffu, sb.w, off);
                    }
                    if (lane < c4n) { const int r = (tid >> 5) * c4n + lane; red[2 * r] = sa; red[2 * r + 1] = sb; }
                    n_rows = 8 * c4n;
                } else {
                    red[2 * tid] = sa; red[2 * tid + 1] = sb;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (tid == 0 && tj == 0) HPF_TL(14);
                if (tid < ((c4n * 2 + 31) & ~31)) {          // whole warps: the swap below is a warp shuffle
                    // threads 2g and 2g+1 add group g's rows of shifted sums and of shifted squares, swap the totals, and store
                    // the tile's mean (from the sums and the group's shift, which thread g keeps: fetched through shared memory)
                    // and the sum of squared deviations from it
                    const int g = tid >> 1, which = tid & 1;
                    const bool mine = tid < c4n * 2;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {                       // n_rows / c4n <= 8
                        const int t2 = g + j * c4n;
                        if (mine && t2 < n_rows) { const float4 v2 = red[2 * t2 + which]; acc.x += v2.x; acc.y += v2.y; acc.z += v2.z; acc.w += v2.w; }
                    }
                    float4 oth;
                    oth.x = __shfl_xor_sync(0xffffffffu, acc.x, 1); oth.y = __shfl_xor_sync(0xffffffffu, acc.y, 1);
                    oth.z = __shfl_xor_sync(0xffffffffu, acc.z, 1); oth.w = __shfl_xor_sync(0xffffffffu, acc.w, 1);
                    const float4 s1 = which ? oth : acc, s2 = which ? acc : oth;
                    const float4 kg = shift_s[mine ? g : 0];
                    const float inv_n = p.stat_inv_tile_rows;       // every tile of a fused launch is full
                    float4 r;
                    if (which == 0) r = make_float4(kg.x + s1.x * inv_n, kg.y + s1.y * inv_n, kg.z + s1.z * inv_n, kg.w + s1.w * inv_n);
                    else r = make_float4(s2.x - s1.x * s1.x * inv_n, s2.y - s1.y * s1.y * inv_n, s2.z - s1.z * s1.z * inv_n, s2.w - s1.w * s1.w * inv_n);
                    if (mine) {
                        float* dstp = p.stat_partials + ((size_t)(tile0 + tj) * 2 + which) * p.c_out + co0 + 4 * g;
                        *reinterpret_cast<float4*>(dstp) = r;
                        if (stat_mode == 1) __threadfence();
                    }
                }
            }
        }
        if (MULTI) asm volatile("bar.sync 1, 256;" ::: "memory");      // the staging area and the row tables serve the next tile
        }   // tiles of this CTA
        {
            const int stat_mode = p.stat_mode;
            if (stat_mode && all_done) {
                // stat_mode 1: the CTA that finishes last turns the per-tile sums into mean and 1/sigma (tiles are added in
                // a fixed order in fp64, so the result does not depend on which CTA that is).  stat_mode 3: the reading
                // convolution adds the few per-tile sums itself, and this kernel ends without a ticket.
                __shared__ int is_last;
                if (stat_mode == 1) asm volatile("bar.sync 1, 256;" ::: "memory");
                if (stat_mode == 1 && tid == 0) {
                    const unsigned int done_before = atomicAdd(p.stat_ticket, 1u);
                    is_last = done_before == vg.x * vg.y - 1;
                }
                if (stat_mode == 1) asm volatile("bar.sync 1, 256;" ::: "memory");
                if (stat_mode == 1 && is_last) {
                    __threadfence();
                    float mu = 0.f, rs = 0.f;
                    // every tile is written out and the pipeline buffers are idle: they hold the reduction
                    bn_combine_partials(p.stat_partials, p.n_tiles, p.c_out, p.stat_inv_rows, p.stat_eps,
                                        reinterpret_cast<float (*)[32][8]>(smem), tid, &mu, &rs);
                    if (tid < p.c_out) { p.stat_out[tid] = mu; p.stat_out[p.c_out + tid] = rs; }
                    if (tid == 0) *p.stat_ticket = 0u;
                }
            }
        }
    }

    if (threadIdx.x == 64) HPF_TL(8);
    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (abort_flag && threadIdx.x == 0) {
        // copies still in flight must land before the shared memory is given back
        for (int it = consumed; it < issued; ++it) {
            const int s = it % p.stages;
            const long long t0 = clock64();
            while (!mbar_try_wait(full0 + 8 * s, (it / p.stages) & 1) && clock64() - t0 < kWaitLimit) {}
        }
    }
    __syncthreads();
    if (!CELL && warp == 0) tmem_dealloc(tmem_base, p.tmem_cols);
    if (threadIdx.x == 0) HPF_TL(9);
#if defined(HPF_TC_TIMELINE) && HPF_TC_TIMELINE == 2
    __syncthreads();
    if (threadIdx.x < 16) {
        const int tiles = vg.x;
        const int cls = (p.R == 3 ? 1 : 0) + 2 * (tiles >= 128 ? 0 : (tiles >= 32 ? 1 : 2)) + (p.bn_in ? 0 : 0);
        if (threadIdx.x == 0) atomicAdd(&g_tl_acc[cls][0], 1ull);
        else if (tl_s[threadIdx.x] > tl_s[0]) atomicAdd(&g_tl_acc[cls][threadIdx.x], tl_s[threadIdx.x] - tl_s[0]);
    }
#endif
    return abort_flag;          // uniform: nobody writes it between the barrier above and the next call's set-up
}

template <bool MULTI, bool KSPLIT = false>
__global__ void __launch_bounds__(320, 2) conv_tc_fwd_kernel(const __grid_constant__ FwdParams gp)
{
    __shared__ FwdScalars p;                 // scalar parameters, see load_scalars
    // Programmatic launch: the next kernel of the stream may be scheduled once every CTA of this one has said so.  Early (here):
    // the successor's set-up hides under this kernel, which shortens a lone stage's chain of kernels.  Late (when the first
    // accumulator is complete, see below): the successor's CTAs do not sit in SM slots for the whole life of this kernel,
    // which is what counts when every stage is busy and slots are what the stages compete for.  The host chooses per launch.
    if (!gp.s.pdl_late) pdl_launch_dependents();
    load_scalars(&p, &gp.s);
    __syncthreads();
    conv_fwd_cta<MULTI ? 1 : (KSPLIT ? 2 : 0)>(&gp, p, make_uint3(blockIdx.x, blockIdx.y, blockIdx.z), make_uint3(gridDim.x, gridDim.y, gridDim.z), 0u, true);
}

// ------------------------------------------------------------------------------------------------
// persistent cell kernel: the forward convolutions of one (partition, micro-batch) cell in ONE resident grid
// ------------------------------------------------------------------------------------------------
// A cell of the pipeline is a chain of a hundred and more small dependent convolutions.  As separate launches each pays
// the launch-to-launch latency, and eight stages' worth of them compete for SM slots in which their CTAs mostly wait.
// Here a fixed, small grid stays resident for the whole cell and walks the list of launches: the CTAs share out the
// CTAs of each launch (virtual CTAs: block index and grid size of the stand-alone launch), run them with the same code,
// and meet at a grid-wide barrier before the next launch, whose input the whole grid has just produced.  Every CTA of
// the grid must be resident at the same time; the host sizes the grids so that all cells that can run concurrently fit
// the GPU together.  The barrier wait is bounded like every other wait here.
struct alignas(64) CellOp {
    FwdParams p;                 // exactly what the stand-alone launch would receive
    unsigned int gx, gy, gz;     // its grid
    unsigned int reserved;
};
struct CellParams {
    const CellOp* ops;           // device memory, written before the launch and read-only for the kernel
    int n_ops;
    unsigned int* barrier;       // {arrivals, generation}: zero before the first use, left with arrivals at zero
    DeviceStatus* status;
    unsigned int tmem_cols;      // the largest accumulator of the list
};

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* ptr)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(unsigned int* ptr, unsigned int v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}

// All CTAs of the grid arrive; the last one opens the next generation.  What the CTAs wrote before the barrier is
// visible to all of them after it, also to copies issued through the async proxy (TMA).  Returns false when the wait ran
// out or another kernel already reported a failure.
__device__ __forceinline__ bool cell_grid_barrier(unsigned int* bar, DeviceStatus* status, int* stop_flag)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int gen = ld_acquire_gpu(bar + 1);      // cannot advance before this CTA has arrived
        __threadfence();
        int stop = 0;
        if (atomicAdd(bar, 1u) == gridDim.x - 1) {
            bar[0] = 0u;
            __threadfence();
            st_release_gpu(bar + 1, gen + 1u);
        } else {
            const long long t0 = clock64();
            int polls = 0;
            while (ld_acquire_gpu(bar + 1) == gen) {
                if ((++polls & 63) == 0 && (clock64() - t0 > kWaitLimit || ld_acquire_gpu(&status->code) != 0u)) { report(status, 9); stop = 1; break; }
            }
        }
        *stop_flag = stop;
    }
    __syncthreads();
    asm volatile("fence.proxy.async;" ::: "memory");
    return *stop_flag == 0;
}

__global__ void __launch_bounds__(320, 2) conv_tc_cell_kernel(const __grid_constant__ CellParams cp)
{
    __shared__ FwdScalars p;
    __shared__ unsigned int vgrid[4];
    __shared__ uint32_t cell_tmem;
    __shared__ int cell_stop;
    constexpr int kWords = (int)(sizeof(FwdScalars) / 4);
    static_assert(sizeof(FwdScalars) % 4 == 0 && kWords + 3 <= 320, "one parameter word per thread");
    const int tid = threadIdx.x;
    if ((tid >> 5) == 0) tmem_alloc(smem_u32(&cell_tmem), cp.tmem_cols);
    if (tid == 0) cell_stop = 0;
    // one word of the parameters per thread: the first launch's now, the next one's while the current one runs
    auto fetch = [&](int op) -> uint32_t {
        const CellOp* o = cp.ops + op;
        if (tid < kWords) return __ldg(reinterpret_cast<const uint32_t*>(&o->p.s) + tid);
        if (tid < kWords + 3) return __ldg(&o->gx + (tid - kWords));
        return 0u;
    };
    uint32_t nxt = fetch(0);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = cell_tmem;
    bool first = true;
    int stop = 0;
    for (int op = 0; op < cp.n_ops && !stop; ++op) {
        if (tid < kWords) reinterpret_cast<uint32_t*>(&p)[tid] = nxt;
        else if (tid < kWords + 3) vgrid[tid - kWords] = nxt;
        if (op + 1 < cp.n_ops) nxt = fetch(op + 1);
        __syncthreads();
        const unsigned int gx = vgrid[0], gy = vgrid[1], gz = vgrid[2], V = gx * gy * gz;
        for (unsigned int v = blockIdx.x; v < V && !stop; v += gridDim.x) {
            const uint3 vb = make_uint3(v % gx, (v / gx) % gy, v / (gx * gy));
            stop = conv_fwd_cta<3>(&cp.ops[op].p, p, vb, make_uint3(gx, gy, gz), tmem_base, first);
            first = false;
        }
        if (stop) break;
        if (op + 1 < cp.n_ops && !cell_grid_barrier(cp.barrier, cp.status, &cell_stop)) stop = 1;
    }
    tc_fence_before();
    __syncthreads();
    if ((tid >> 5) == 0) tmem_dealloc(tmem_base, cp.tmem_cols);
}

// ------------------------------------------------------------------------------------------------
// weight-gradient kernel: 6 warps = TMA producer, MMA issuer, 4 transposer / epilogue warps
// ------------------------------------------------------------------------------------------------
// raw [rows][channels] (dense) -> K-major: channel rows of 128 bytes (32 pixels), 16-byte chunks XOR-swizzled by
// (row % 8), further groups of 32 pixels `atom_stride` bytes apart.  With SPLIT the hi part goes to dst and the
// lo part to dst_lo.  128 threads; per 4 pixels a thread issues 4 conflict-free 32-bit loads and one (two)
// conflict-free 128-bit store(s).
template <bool SPLIT>
__device__ __forceinline__ void transpose_tile(const uint8_t* raw, uint8_t* dst, uint8_t* dst_lo, int channels, int rows,
                                               uint32_t atom_stride, int tid)
{
    const int items = channels * (rows >> 2);
    const bool pow2 = (channels & (channels - 1)) == 0;
    const int shift = 31 - __clz(channels);
    for (int it = tid; it < items; it += 128) {
        const int c = pow2 ? (it & (channels - 1)) : (it % channels);
        const int p4 = pow2 ? (it >> shift) : (it / channels);
        const float* src = reinterpret_cast<const float*>(raw) + (p4 * 4) * channels + c;
        float4 v;
        v.x = src[0]; v.y = src[channels]; v.z = src[2 * channels]; v.w = src[3 * channels];
        const uint32_t o = (uint32_t)(p4 >> 3) * atom_stride + (uint32_t)c * 128u + (uint32_t)(((p4 & 7) ^ (c & 7)) << 4);
        if (SPLIT) {
            const float4 h = make_float4(tf32_hi(v.x), tf32_hi(v.y), tf32_hi(v.z), tf32_hi(v.w));
            *reinterpret_cast<float4*>(dst + o) = h;
            *reinterpret_cast<float4*>(dst_lo + o) = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
        } else {
            *reinterpret_cast<float4*>(dst + o) = v;
        }
    }
}

__global__ void __launch_bounds__(192) conv_tc_wgrad_kernel(const __grid_constant__ WgradParams gp)
{
    __shared__ WgradScalars p;                 // scalar parameters, see load_scalars
    pdl_launch_dependents();
    load_scalars(&p, &gp.s);
    __syncthreads();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[4 * 4 + 1];       // full_raw[4], empty_raw[4], full_t[4], empty_t[4], accum
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued, raw_consumed;

    const uint32_t base_off = ((smem_u32(smem_raw) + 1023u) & ~1023u) - smem_u32(smem_raw);
    uint8_t* smem = smem_raw + base_off;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full_raw0 = smem_u32(&bars[0]), empty_raw0 = smem_u32(&bars[4]), full_t0 = smem_u32(&bars[8]),
                   empty_t0 = smem_u32(&bars[12]), accum_bar = smem_u32(&bars[16]);
    // shared memory: raw stages first, then the transposed stages
    const uint32_t t_region0 = (uint32_t)p.raw_stages * p.raw_bytes;

    const int split = blockIdx.x;
    const int tap0 = blockIdx.y * p.taps_per_cta;
    const int m_chunks = p.c_out / p.m_chunk;
    const int m0 = (blockIdx.z % m_chunks) * p.m_chunk;
    const int cn0 = (blockIdx.z / m_chunks) * p.n_cols;
    int ntaps = p.R * p.R - tap0;
    if (ntaps > p.taps_per_cta) ntaps = p.taps_per_cta;
    const int tile_begin = split * p.tiles_per_split;
    int tile_end = tile_begin + p.tiles_per_split;
    if (tile_end > p.n_tiles) tile_end = p.n_tiles;
    const int total = tile_end - tile_begin;
    const int katoms = p.rows >> 5;
    const uint32_t raw_a = (uint32_t)p.rows * p.m_chunk * 4u, raw_b = (uint32_t)p.rows * p.n_cols * 4u;
    // The transposed dy operand keeps only its m_chunk channel rows per pixel group.  An MMA always reads 128 rows from
    // the operand's base: the rows beyond m_chunk come from whatever follows in shared memory (the other operand, the
    // next stage, the slack after the last stage) and land in accumulator lanes that the epilogue never reads.
    const uint32_t a_atom = (uint32_t)p.m_chunk * 128u;                   // one pixel group of the dy operand
    const uint32_t t_a = (uint32_t)katoms * a_atom;
    // transposed B: [pixel group of 32][tap][input channel] rows of 128 bytes, so that consecutive taps are consecutive
    // N rows of one operand and one MMA covers several taps at once
    const uint32_t t_b_tap = (uint32_t)p.n_cols * 128u;                   // one tap inside one pixel group
    const uint32_t t_b_atom = (uint32_t)p.taps_per_cta * t_b_tap;         // one pixel group, all taps
    // transposed stage layout: A_hi | B_hi | A_lo | B_lo
    const uint32_t t_half = t_a + (uint32_t)katoms * t_b_atom;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 4; ++s) {
            mbar_init(full_raw0 + 8 * s, 1); mbar_init(empty_raw0 + 8 * s, 4);
            mbar_init(full_t0 + 8 * s, 4); mbar_init(empty_t0 + 8 * s, 1);
        }
        mbar_init(accum_bar, 1);
        abort_flag = 0; issued = 0; raw_consumed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), p.tmem_cols);
    if (p.box_rows < p.rows) {
        // A pixel box whose size is not a multiple of 32 leaves the last rows of every raw tile untouched by the
        // copies: they are zeroed once and add nothing to the sums over pixels.
        const int pad_rows = p.rows - p.box_rows;
        for (int s = 0; s < p.raw_stages; ++s) {
            float* st = reinterpret_cast<float*>(smem + s * p.raw_bytes);
            for (int i = threadIdx.x; i < pad_rows * p.m_chunk; i += blockDim.x) st[p.box_rows * p.m_chunk + i] = 0.f;
            for (int tp = 0; tp < ntaps; ++tp) {
                float* bt = reinterpret_cast<float*>(smem + s * p.raw_bytes + raw_a + tp * raw_b);
                for (int i = threadIdx.x; i < pad_rows * p.n_cols; i += blockDim.x) bt[p.box_rows * p.n_cols + i] = 0.f;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();              // everything above touched only parameters, shared and tensor memory
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            // no division in the loop: the stage, its parity, the tile's position and the taps' offsets are counters
            const int raw_stages = p.raw_stages, tiles_w = p.tiles_w, tiles_h = p.tiles_h, R = p.R, pad = p.pad;
            const int box_w = p.box_w, box_h = p.box_h, box_n = p.box_n;
            const uint32_t raw_bytes = p.raw_bytes, tx = p.tx_a + (uint32_t)ntaps * p.tx_per_tap;
            int tw, th, tn;
            { int t = tile_begin; tw = t % tiles_w; t /= tiles_w; th = t % tiles_h; tn = t / tiles_h; }
            const int r_first = tap0 / R, sx_first = tap0 - r_first * R;
            int it = 0, s = 0;
            uint32_t par = 1u;
            for (; it < total; ++it) {
                if (!mbar_wait(empty_raw0 + 8 * s, par, &abort_flag)) { report(p.status, 3); break; }
                const int q0 = tw * box_w, p0 = th * box_h, n0 = tn * box_n;
                const uint32_t dst = smem_base + s * raw_bytes;
                const uint32_t bar = full_raw0 + 8 * s;
                mbar_expect_tx(bar, tx);
                tma_load_4d(dst, &gp.tm_a, bar, m0, q0, p0, n0);
                int r = r_first, sx = sx_first;
                for (int tp = 0; tp < ntaps; ++tp) {
                    tma_load_4d(dst + raw_a + tp * raw_b, &gp.tm_b, bar, cn0, q0 + sx - pad, p0 + r - pad, n0);
                    if (++sx == R) { sx = 0; ++r; }
                }
                if (++tw == tiles_w) { tw = 0; if (++th == tiles_h) { th = 0; ++tn; } }
                if (++s == raw_stages) { s = 0; par ^= 1u; }
            }
            issued = it;
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            const int t_stages = p.t_stages;
            int it = 0, t = 0;
            uint32_t tpar = 0;
            for (; it < total; ++it) {
                if (!mbar_wait(full_t0 + 8 * t, tpar, &abort_flag)) { report(p.status, 4); break; }
                tc_fence_after();
                const uint32_t a_src = smem_base + t_region0 + t * p.t_bytes, b_src = a_src + t_a;
                // taps are stacked along N: groups of up to 256 / n_cols taps per MMA
                for (int tg = 0; tg < ntaps; tg += p.taps_per_mma) {
                    const int nt = ntaps - tg < p.taps_per_mma ? ntaps - tg : p.taps_per_mma;
                    const uint32_t idesc = nt == p.taps_per_mma ? p.idesc : p.idesc_tail;
                    const uint32_t acc = tmem_base + (uint32_t)(tg * p.n_cols);
                    for (int kb = 0; kb < katoms; ++kb)
                        for (int k8 = 0; k8 < 4; ++k8) {
                            const uint32_t ao = (uint32_t)kb * a_atom + 32u * k8;
                            const uint32_t bo = (uint32_t)kb * t_b_atom + (uint32_t)tg * t_b_tap + 32u * k8;
                            const uint64_t ad = smem_desc(a_src + ao, 16, 1024, 128);
                            const uint64_t bd = smem_desc(b_src + bo, 16, 1024, 128);
                            umma_tf32(acc, ad, bd, idesc, (it | kb | k8) ? 1u : 0u);
                            if (p.passes == 3) {
                                const uint64_t adl = smem_desc(a_src + t_half + ao, 16, 1024, 128);
                                const uint64_t bdl = smem_desc(b_src + t_half + bo, 16, 1024, 128);
                                umma_tf32(acc, adl, bd, idesc, 1u);
                                umma_tf32(acc, ad, bdl, idesc, 1u);
                            }
                        }
                }
                umma_commit(empty_t0 + 8 * t);
                if (++t == t_stages) { t = 0; tpar ^= 1u; }
            }
            if (it == total) umma_commit(accum_bar);
        }
    } else {
        // ---- transposers (warps 2..5), then the epilogue ----
        const int tid = threadIdx.x - 64;
        int it = 0, s = 0, t = 0;
        uint32_t spar = 0, tpar = 1u;
        const int raw_stages = p.raw_stages, t_stages = p.t_stages;
        bool ok = true;
        for (; it < total && ok; ++it) {
            ok = mbar_wait(full_raw0 + 8 * s, spar, &abort_flag) &&
                 mbar_wait(empty_t0 + 8 * t, tpar, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { if (lane == 0) report(p.status, 5); break; }
            const uint8_t* raw = smem + s * p.raw_bytes;
            uint8_t* tdst = smem + t_region0 + t * p.t_bytes;
            if (p.passes == 3) {
                transpose_tile<true>(raw, tdst, tdst + t_half, p.m_chunk, p.rows, a_atom, tid);
                for (int tp = 0; tp < ntaps; ++tp)
                    transpose_tile<true>(raw + raw_a + tp * raw_b, tdst + t_a + tp * t_b_tap, tdst + t_half + t_a + tp * t_b_tap,
                                         p.n_cols, p.rows, t_b_atom, tid);
            } else {
                transpose_tile<false>(raw, tdst, nullptr, p.m_chunk, p.rows, a_atom, tid);
                for (int tp = 0; tp < ntaps; ++tp)
                    transpose_tile<false>(raw + raw_a + tp * raw_b, tdst + t_a + tp * t_b_tap, nullptr, p.n_cols, p.rows, t_b_atom, tid);
            }
            fence_async_smem();     // generic-proxy writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) { mbar_arrive(full_t0 + 8 * t); mbar_arrive(empty_raw0 + 8 * s); }
            if (++s == raw_stages) { s = 0; spar ^= 1u; }
            if (++t == t_stages) { t = 0; tpar ^= 1u; }
        }
        if (tid == 0) raw_consumed = it;

        bool done = ok && mbar_wait(accum_bar, 0, &abort_flag);
        done = __all_sync(0xffffffffu, done);
        if (done) {
            tc_fence_after();
            const int row = (warp & 3) * 32 + lane;          // TMEM lane = output channel within the chunk
            const bool valid = row < p.m_chunk;
            const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
            float* obase = p.out + (long long)split * p.split_stride + ((long long)(m0 + row) * p.R * p.R) * p.c_in + cn0;
            for (int tp = 0; tp < ntaps; ++tp)
                for (int c0 = 0; c0 < p.n_cols; c0 += 16) {
                    float v[16];
                    tmem_ld16(lane_addr + (uint32_t)(tp * p.n_cols + c0), v);
                    if (valid) {
                        // a gradient slot starts at m*G floats: 16-byte aligned only if G is a multiple of 4
                        float* o = obase + (long long)(tap0 + tp) * p.c_in + c0;
                        if ((reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j) o[j] = v[j];
                        }
                    }
                }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (abort_flag && threadIdx.x == 0) {
        for (int it = raw_consumed; it < issued; ++it) {
            const int s = it % p.raw_stages;
            const long long t0 = clock64();
            while (!mbar_try_wait(full_raw0 + 8 * s, (it / p.raw_stages) & 1) && clock64() - t0 < kWaitLimit) {}
        }
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, p.tmem_cols);
}

// ------------------------------------------------------------------------------------------------
// weight-gradient kernel without the transposition: the tensor core reads the TMA tiles as they land
// ------------------------------------------------------------------------------------------------
// dW[co][tap][ci] = sum over pixels of dy[pixel][co] * x[pixel + tap][ci]: the reduction runs over pixels, and both
// tensors keep channels innermost in memory, so both operands are MN-major.  A TMA box of 32 channels x `rows` pixels with
// the 32-byte-atom swizzle is exactly the tile the tensor core wants (smem_desc_mn): 6 warps = TMA producer, MMA issuer and
// 4 warps that only read the accumulators at the end (with three passes they also write every tile's lo part, position
// by position - no transposition either).  A 16-channel tensor is copied with 16-channel boxes: the
// copy still gives every pixel a 128-byte row and leaves its second half alone; those columns and lanes of the
// accumulator hold products of whatever the shared memory held and are never read.  An MMA always reads 128 operand
// rows = 4 blocks from the dy tile's base: blocks beyond the tile's own are the x tile or what follows it, and land in
// accumulator lanes nobody reads.
__global__ void __launch_bounds__(192) conv_tc_wgrad_direct_kernel(const __grid_constant__ WgradDirectParams gp)
{
    __shared__ WgradDirectScalars p;
    pdl_launch_dependents();
    load_scalars(&p, &gp.s);
    __syncthreads();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[3 * 8 + 1];       // full[8], empty[8], split[8], accum
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued, consumed;

    const uint32_t base_off = ((smem_u32(smem_raw) + 1023u) & ~1023u) - smem_u32(smem_raw);
    uint8_t* smem = smem_raw + base_off;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[8]), split0 = smem_u32(&bars[16]), accum_bar = smem_u32(&bars[24]);

    const int split = blockIdx.x;
    const int tap0 = blockIdx.y * p.taps_per_cta;
    const int m_chunks = p.c_out / p.m_chunk;
    const int m0 = (blockIdx.z % m_chunks) * p.m_chunk;
    const int cn0 = (blockIdx.z / m_chunks) * p.n_cols;
    int ntaps = p.R * p.R - tap0;
    if (ntaps > p.taps_per_cta) ntaps = p.taps_per_cta;
    const int tile_begin = split * p.tiles_per_split;
    int tile_end = tile_begin + p.tiles_per_split;
    if (tile_end > p.n_tiles) tile_end = p.n_tiles;
    const int total = tile_end - tile_begin;
    const uint32_t block_bytes = (uint32_t)p.rows * 128u;                 // one 32-channel block of a tile
    const uint32_t a_bytes = (uint32_t)p.m_blocks * block_bytes;          // the dy tile
    const uint32_t tap_bytes = (uint32_t)p.n_blocks * block_bytes;        // one tap's x tile
    const int slot = p.n_blocks * 32;                                     // accumulator columns of one tap

    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); mbar_init(split0 + 8 * s, 4); }
        mbar_init(accum_bar, 1);
        abort_flag = 0; issued = 0; consumed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), p.tmem_cols);
    if (p.box_rows < p.rows) {
        // A pixel box that is not a multiple of 8 pixels leaves the last rows of every block untouched by the copies:
        // zeroed once, they add nothing to the sums over pixels.
        const int pad_rows = p.rows - p.box_rows;
        const int blocks = p.m_blocks + ntaps * p.n_blocks;
        for (int s = 0; s < p.stages; ++s)
            for (int part = 0; part < (p.passes == 3 ? 2 : 1); ++part)
                for (int b = 0; b < blocks; ++b) {
                    float* blk = reinterpret_cast<float*>(smem + s * p.stage_bytes + part * p.lo_off + b * block_bytes) + p.box_rows * 32;
                    for (int i = threadIdx.x; i < pad_rows * 32; i += blockDim.x) blk[i] = 0.f;
                }
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();              // everything above touched only parameters, shared and tensor memory
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            const int stages = p.stages, tiles_w = p.tiles_w, tiles_h = p.tiles_h, R = p.R, pad = p.pad;
            const int box_w = p.box_w, box_h = p.box_h, box_n = p.box_n, m_blocks = p.m_blocks, n_blocks = p.n_blocks;
            const int m_box = p.m_box, n_box = p.n_box;
            const uint32_t stage_bytes = p.stage_bytes, tx = p.tx_bytes_a + (uint32_t)ntaps * p.tx_per_tap;
            int tw, th, tn;
            { int t = tile_begin; tw = t % tiles_w; t /= tiles_w; th = t % tiles_h; tn = t / tiles_h; }
            const int r_first = tap0 / R, sx_first = tap0 - r_first * R;
            int it = 0, s = 0;
            uint32_t par = 1u;
            for (; it < total; ++it) {
                if (!mbar_wait(empty0 + 8 * s, par, &abort_flag)) { report(p.status, 3); break; }
                const int q0 = tw * box_w, p0 = th * box_h, n0 = tn * box_n;
                uint32_t dst = smem_base + s * stage_bytes;
                const uint32_t bar = full0 + 8 * s;
                mbar_expect_tx(bar, tx);
                for (int b = 0; b < m_blocks; ++b, dst += block_bytes) tma_load_4d(dst, &gp.tm_a, bar, m0 + b * m_box, q0, p0, n0);
                int r = r_first, sx = sx_first;
                for (int tp = 0; tp < ntaps; ++tp) {
                    for (int b = 0; b < n_blocks; ++b, dst += block_bytes)
                        tma_load_4d(dst, &gp.tm_b, bar, cn0 + b * n_box, q0 + sx - pad, p0 + r - pad, n0);
                    if (++sx == R) { sx = 0; ++r; }
                }
                if (++tw == tiles_w) { tw = 0; if (++th == tiles_h) { th = 0; ++tn; } }
                if (++s == stages) { s = 0; par ^= 1u; }
            }
            issued = it;
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            const int stages = p.stages, k8n = p.rows >> 3;
            const bool three = p.passes == 3;
            const uint32_t ready0 = three ? split0 : full0;
            int it = 0, s = 0;
            uint32_t par = 0;
            for (; it < total; ++it) {
                if (!mbar_wait(ready0 + 8 * s, par, &abort_flag)) { report(p.status, 4); break; }
                tc_fence_after();
                const uint32_t a_src = smem_base + s * p.stage_bytes, b_src = a_src + a_bytes;
                // taps are consecutive blocks of the x operand: groups of up to 256 accumulator columns per MMA
                for (int tg = 0; tg < ntaps; tg += p.taps_per_mma) {
                    const int nt = ntaps - tg < p.taps_per_mma ? ntaps - tg : p.taps_per_mma;
                    const uint32_t idesc = nt == p.taps_per_mma ? p.idesc : p.idesc_tail;
                    const uint32_t acc = tmem_base + (uint32_t)(tg * slot);
                    const uint32_t b_tg = b_src + (uint32_t)tg * tap_bytes;
                    for (int k8 = 0; k8 < k8n; ++k8) {
                        const uint64_t ad = smem_desc_mn(a_src + 1024u * k8, block_bytes);
                        const uint64_t bd = smem_desc_mn(b_tg + 1024u * k8, block_bytes);
                        umma_tf32(acc, ad, bd, idesc, (it | k8) ? 1u : 0u);
                        if (three) {
                            const uint64_t adl = smem_desc_mn(a_src + p.lo_off + 1024u * k8, block_bytes);
                            const uint64_t bdl = smem_desc_mn(b_tg + p.lo_off + 1024u * k8, block_bytes);
                            umma_tf32(acc, adl, bd, idesc, 1u);
                            umma_tf32(acc, ad, bdl, idesc, 1u);
                        }
                    }
                }
                umma_commit(empty0 + 8 * s);
                if (++s == stages) { s = 0; par ^= 1u; }
            }
            if (!three) consumed = it;
            if (it == total) umma_commit(accum_bar);
        }
    } else {
        const int tid = threadIdx.x - 64;
        bool ok = true;
        if (p.passes == 3) {
            // ---- splitters: the tile stays where the copy put it, its lo part goes to the stage's second half, same position ----
            const int stages = p.stages;
            // 16-byte pieces of the dy tile and of the x tiles.  A tile of a 16-channel tensor holds data in one half of
            // every 128-byte row only (which half: bit 1 of the row number, the swizzle's doing): 4 pieces per row then.
            const int a_half = p.m_box == 16, b_half = p.n_box == 16;
            const int a4 = (int)(a_bytes >> 4) >> a_half;
            const int n4 = a4 + ((int)(((uint32_t)(ntaps * p.n_blocks) * block_bytes) >> 4) >> b_half);
            int it = 0, s = 0;
            uint32_t par = 0;
            for (; it < total && ok; ++it) {
                ok = mbar_wait(full0 + 8 * s, par, &abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) report(p.status, 5); break; }
                float4* hi = reinterpret_cast<float4*>(smem + s * p.stage_bytes);
                float4* lo = reinterpret_cast<float4*>(smem + s * p.stage_bytes + p.lo_off);
                for (int i = tid; i < n4; i += 128) {
                    int j;                                  // the piece's place among the stage's 16-byte pieces
                    if (i < a4) j = a_half ? ((i >> 2) << 3) + ((i >> 3) & 1) * 4 + (i & 3) : i;
                    else {
                        const int k = i - a4;
                        j = (int)(a_bytes >> 4) + (b_half ? ((k >> 2) << 3) + ((k >> 3) & 1) * 4 + (k & 3) : k);
                    }
                    // the tile stays as copied: the tensor core's truncation of a 32-bit operand is the hi part
                    const float4 v = hi[j];
                    const float4 h = make_float4(tf32_hi(v.x), tf32_hi(v.y), tf32_hi(v.z), tf32_hi(v.w));
                    lo[j] = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
                }
                fence_async_smem();     // generic-proxy writes -> tensor-core reads
                __syncwarp();
                if (lane == 0) mbar_arrive(split0 + 8 * s);
                if (++s == stages) { s = 0; par ^= 1u; }
            }
            if (tid == 0) consumed = it;
        }
        // ---- epilogue ----
        bool done = ok && mbar_wait(accum_bar, 0, &abort_flag);
        done = __all_sync(0xffffffffu, done);
        if (done) {
            tc_fence_after();
            const int row = (warp & 3) * 32 + lane;          // TMEM lane = output channel within the chunk
            const bool valid = row < p.m_chunk;
            const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
            float* obase = p.out + (long long)split * p.split_stride + ((long long)(m0 + row) * p.R * p.R) * p.c_in + cn0;
            if ((warp & 3) * 32 < p.m_chunk)                 // a whole warp of lanes beyond the chunk has nothing to read
                for (int tp = 0; tp < ntaps; ++tp)
                    for (int c0 = 0; c0 < p.n_cols; c0 += 16) {
                        float v[16];
                        tmem_ld16(lane_addr + (uint32_t)(tp * slot + c0), v);
                        if (valid) {
                            // a gradient slot starts at m*G floats: 16-byte aligned only if G is a multiple of 4
                            float* o = obase + (long long)(tap0 + tp) * p.c_in + c0;
                            if ((reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
#pragma unroll
                                for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 16; ++j) o[j] = v[j];
                            }
                        }
                    }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (abort_flag && threadIdx.x == 0) {
        // copies in flight must land before the shared memory is given back
        for (int it = consumed; it < issued; ++it) {
            const int s = it % p.stages;
            const long long t0 = clock64();
            while (!mbar_try_wait(full0 + 8 * s, (it / p.stages) & 1) && clock64() - t0 < kWaitLimit) {}
        }
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, p.tmem_cols);
}

// dw[i] = sum over splits of partials[z][i], in an order fixed by the launch shape: thread (lane, zl) adds the
// splits zl, zl+8, ... ascending, then the 8 partial sums are added ascending.  32 float4 per block.
__global__ void __launch_bounds__(256)
wgrad_partials_reduce_kernel(const float* __restrict__ partials, float* __restrict__ dw, long long n, int splits)
{
    __shared__ float4 sh[8][32];
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31, zl = threadIdx.x >> 5;
    const long long n4 = n / 4;          // n is a multiple of 4 and the partials are 16-byte aligned; dw may not be
    const long long i = (long long)blockIdx.x * 32 + lane;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < n4) {
        // four splits per batch, the four loads in flight together; splits beyond the last add zero
        for (int z0 = zl; z0 < splits; z0 += 32) {
            float4 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int z = z0 + 8 * j;
                v[j] = z < splits ? __ldcg(reinterpret_cast<const float4*>(partials + (long long)z * n) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) { s.x += v[j].x; s.y += v[j].y; s.z += v[j].z; s.w += v[j].w; }
        }
    }
    sh[zl][lane] = s;
    __syncthreads();
    if (zl == 0 && i < n4) {
        for (int k = 1; k < 8; ++k) { const float4 v = sh[k][lane]; s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
        if ((reinterpret_cast<uintptr_t>(dw) & 15u) == 0) reinterpret_cast<float4*>(dw)[i] = s;
        else { dw[4 * i] = s.x; dw[4 * i + 1] = s.y; dw[4 * i + 2] = s.z; dw[4 * i + 3] = s.w; }
    }
}

// Weight preparation, once per step: for every convolution of the table (or the one passed by value), the hi / lo split of the weights
// ([K][R][R][C], forward operand) and of the weights rearranged for the data gradient
// (wt[c][R-1-r][R-1-s][k] = w[k][r][s][c]).  blockIdx.x = table entry; blockIdx.y strides over 32 x 32 tiles of the (k, c)
// matrix of one filter tap, transposed through shared memory so that reads and all four writes are coalesced.
__device__ __forceinline__ void weight_prep_one(const float* __restrict__ params, float* __restrict__ w_hi, float* __restrict__ w_lo,
                                                float* __restrict__ wt_hi, float* __restrict__ wt_lo, const WeightPrepEntry e)
{
    __shared__ float sm[32][33];
    const int C = e.C, K = e.K, R = e.R;
    const int ct = (C + 31) / 32, kt = (K + 31) / 32;
    const int n_tiles = R * R * ct * kt;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8 threads
    const float* w = params + e.w_off;
    for (int tile = blockIdx.y; tile < n_tiles; tile += gridDim.y) {
        const int rs = tile / (ct * kt), rem = tile % (ct * kt);
        const int k0 = (rem / ct) * 32, c0 = (rem % ct) * 32;
        const int r = rs / R, s2 = rs % R;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = k0 + ty + 8 * j, c = c0 + tx;
            if (k < K && c < C) {
                const long long src = (((long long)k * R + r) * R + s2) * C + c;
                const float v = __ldg(&w[src]);
                const float h = tf32_hi(v);
                w_hi[e.w_off + src] = h; w_lo[e.w_off + src] = v - h;
                sm[ty + 8 * j][tx] = v;
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + ty + 8 * j, k = k0 + tx;
            if (c < C && k < K) {
                const float v = sm[tx][ty + 8 * j];
                const float h = tf32_hi(v);
                const long long dst = (((long long)c * R + (R - 1 - r)) * R + (R - 1 - s2)) * K + k;
                wt_hi[e.w_off + dst] = h; wt_lo[e.w_off + dst] = v - h;
            }
        }
        __syncthreads();
    }
}
__global__ void __launch_bounds__(256)
weight_prep_kernel(const float* __restrict__ params, float* __restrict__ w_hi, float* __restrict__ w_lo,
                   float* __restrict__ wt_hi, float* __restrict__ wt_lo, const WeightPrepEntry* __restrict__ table)
{
    weight_prep_one(params, w_hi, w_lo, wt_hi, wt_lo, table[blockIdx.x]);
}
__global__ void __launch_bounds__(256)
weight_prep_single_kernel(const float* __restrict__ w, float* __restrict__ w_hi, float* __restrict__ w_lo,
                          float* __restrict__ wt_hi, float* __restrict__ wt_lo, WeightPrepEntry e)
{
    weight_prep_one(w, w_hi, w_lo, wt_hi, wt_lo, e);
}

// ------------------------------------------------------------------------------------------------
// host: tile geometry and tensor maps
// ------------------------------------------------------------------------------------------------
struct PixelBox { int w, h, n, rows; };

// A rectangular box of output pixels with at most `max_rows` pixels: all of w (or, for maps wider than a tile, a
// divisor of w), then rows of h, then images.
bool choose_box(int Q, int P, int N, int max_rows, int rows_mult, PixelBox* out)
{
    PixelBox b;
    if (Q > max_rows) {
        // a row of the map does not fit one tile: the widest divisor of the row that does
        int w = 0;
        for (int d = max_rows; d >= 4 && !w; --d)
            if (Q % d == 0 && (rows_mult <= 1 || d % rows_mult == 0)) w = d;
        if (!w) return false;
        b.w = w; b.h = 1; b.n = 1; b.rows = w;
        *out = b;
        return true;
    }
    b.w = Q;
    int hmax = max_rows / Q;
    if (hmax > P) hmax = P;
    b.h = 1;
    for (int h = hmax; h >= 1; --h)
        if (P % h == 0) { b.h = h; break; }
    // prefer a non-dividing taller box when the dividing one wastes more than half of the tile
    if (b.h * 2 <= hmax && rows_mult <= 1) b.h = hmax;
    b.n = 1;
    if (b.h == P) {
        int nmax = max_rows / (Q * P);
        if (nmax > N) nmax = N;
        if (nmax >= 1) b.n = nmax;
    }
    b.rows = b.w * b.h * b.n;
    if (rows_mult > 1 && b.rows % rows_mult) {
        // shrink until the row count is a multiple of rows_mult
        bool found = false;
        for (int n = b.n; n >= 1 && !found; --n)
            for (int h = b.h; h >= 1 && !found; --h)
                if ((Q * h * n) % rows_mult == 0 && (n == 1 || h == P)) { b.h = h; b.n = n; found = true; }
        if (!found) return false;
        b.rows = b.w * b.h * b.n;
    }
    *out = b;
    return true;
}

int chunk_of(int channels) { return channels % 32 == 0 ? 32 : 16; }
unsigned int pow2_cols(int need)
{
    unsigned int c = 32;
    while ((int)c < need) c <<= 1;
    return c;
}

// Geometry of the forward pass and of the data gradient seen as a forward-like problem.
struct FwdView {
    int N, P, Q;          // output pixel grid
    int c_in, c_out;      // reduction channels, output channels
    int R, pad;           // taps and tap shift
    int in_w, in_h;       // extent of the input tensor map's pixel dims
    long long in_sw, in_sh, in_sn;   // input strides (floats) of the tensor map's w, h, n dims
    long long os_n, os_h, os_w, dense_h, dense_w;
    int zero_fill, out_h, out_w;
};

bool fwd_view(const ConvShape& s, int pass, FwdView* v)
{
    if (s.C % 16 || s.K % 16) return false;
    if (s.R != 1 && s.R != 3) return false;
    if (s.R == 3 && (s.stride != 1 || s.pad != 1)) return false;
    if (s.R == 1 && s.pad != 0) return false;
    if (s.stride < 1 || s.stride > 2) return false;
    if (pass == PASS_FWD) {
        v->N = s.N; v->P = s.P; v->Q = s.Q; v->c_in = s.C; v->c_out = s.K; v->R = s.R; v->pad = s.pad;
        v->in_w = s.stride == 1 ? s.W : s.Q; v->in_h = s.stride == 1 ? s.H : s.P;
        v->in_sw = (long long)s.stride * s.C; v->in_sh = (long long)s.stride * s.W * s.C; v->in_sn = (long long)s.H * s.W * s.C;
        v->os_w = s.K; v->os_h = (long long)s.Q * s.K; v->os_n = (long long)s.P * s.Q * s.K;
        v->dense_h = v->os_h; v->dense_w = v->os_w; v->zero_fill = 1; v->out_h = s.P; v->out_w = s.Q;
    } else {
        // dx = "forward" convolution of dy with the rearranged weights; tap shift R-1-pad
        v->N = s.N; v->P = s.stride == 1 ? s.H : s.P; v->Q = s.stride == 1 ? s.W : s.Q;
        v->c_in = s.K; v->c_out = s.C; v->R = s.R; v->pad = s.R - 1 - s.pad;
        v->in_w = s.Q; v->in_h = s.P;
        v->in_sw = s.K; v->in_sh = (long long)s.Q * s.K; v->in_sn = (long long)s.P * s.Q * s.K;
        v->dense_w = s.C; v->dense_h = (long long)s.W * s.C;
        v->os_w = (long long)s.stride * s.C; v->os_h = (long long)s.stride * s.W * s.C; v->os_n = (long long)s.H * s.W * s.C;
        v->zero_fill = s.stride; v->out_h = s.H; v->out_w = s.W;
    }
    if (v->c_out > 256 && v->c_out % 256) return false;
    return true;
}

constexpr int kSwizzle128Atom32 = 1;      // encode(): rows of 128 bytes, 32-byte chunks XOR-swizzled by (row % 4)
cudaError_t encode(CUtensorMap* tm, const float* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                   const cuuint32_t* box, int swizzle_bytes)
{
    if (!g_encode) return cudaErrorNotReady;
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<float*>(base), dims, strides_bytes, box,
                          ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : (swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                             : (swizzle_bytes == kSwizzle128Atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_NONE)),
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// How many pixel splits (CTAs along x) a weight-gradient launch of n_tiles pixel tiles gets.
void wgrad_splits(const ConvShape& s, int n_tiles, int ctas_per_split, int max_ctas, int* splits_out, int* tiles_per_split_out)
{
    const int taps = s.R * s.R;
    // enough CTAs to spread the pixel walk, few enough that the partials stay a fraction of the operand bytes
    const double operand_bytes = 4.0 * ((double)s.N * s.P * s.Q * s.K + (double)s.N * s.P * s.Q * s.C);
    const double dw_bytes = 4.0 * (double)s.K * taps * s.C;
    int splits = n_tiles / 4;
    int cap = (int)(operand_bytes / (4.0 * dw_bytes));
    // small problems are latency bound, not byte bound: spread the pixel walk over several dozen CTAs
    const int want = (kWgradWantCtas + ctas_per_split - 1) / ctas_per_split;
    if (cap < want) cap = want;
    if (splits > cap) splits = cap;
    if (splits > 296) splits = 296;          // two CTAs per SM
    if (max_ctas > 0) {
        // the caller wants the launch to take little SM time (CTAs x (fixed cost + tiles)) rather than to be short
        int ms = max_ctas / ctas_per_split;
        if (ms < 1) ms = 1;
        if (splits > ms) splits = ms;
    }
    if (splits > n_tiles / 2) splits = n_tiles / 2;
    if (splits < 1) splits = 1;
    *tiles_per_split_out = (n_tiles + splits - 1) / splits;
    *splits_out = (n_tiles + *tiles_per_split_out - 1) / *tiles_per_split_out;
}

struct WgradGeom {
    PixelBox box;
    int m_chunk, n_cols, taps_per_cta, tap_groups, raw_stages, t_stages, splits, tiles_per_split, n_tiles, rows_padded;
    unsigned int raw_bytes, t_bytes, tmem_cols;
};

bool wgrad_geom(const ConvShape& s, int passes, WgradGeom* g, int max_ctas = 0)
{
    if (s.C % 16 || s.K % 16) return false;
    if (s.R != 1 && s.R != 3) return false;
    if (s.R == 3 && (s.stride != 1 || s.pad != 1)) return false;
    if (s.R == 1 && s.pad != 0) return false;
    if (s.stride < 1 || s.stride > 2) return false;
    g->m_chunk = s.K < 128 ? s.K : 128;
    if (s.K % g->m_chunk) return false;
    const int taps = s.R * s.R;
    const unsigned int parts = passes == 3 ? 2u : 1u;
    // input channels per CTA (all up to 256, else 128 or 64), taps per CTA (all, one row of the window, or one)
    // and pixels per tile (64 or 32): the first combination whose accumulators fit tensor memory and whose
    // 2 raw + 2 transposed stages fit shared memory
    bool found = false;
    const int ncand[3] = {s.C < 256 ? s.C : 256, 128, 64};
    const int cand[3] = {taps, taps == 9 ? 3 : 1, 1};
    for (int ni = 0; ni < 3 && !found; ++ni) {
        const int n_cols = ncand[ni];
        if (n_cols > s.C || s.C % n_cols || (ni > 0 && n_cols >= ncand[0])) continue;
        for (int ci = 0; ci < 3 && !found; ++ci) {
            const int tpc = cand[ci];
            if (tpc * n_cols > 512) continue;
            for (int rows = 64; rows >= 32 && !found; rows >>= 1) {
                PixelBox b;
                if (!choose_box(s.Q, s.P, s.N, rows, 1, &b)) continue;
                const int padded = (b.rows + 31) / 32 * 32;       // shared-memory rows: whole groups of 32 pixels
                const unsigned int raw = (unsigned int)padded * 4u * (unsigned int)(g->m_chunk + tpc * n_cols);
                const unsigned int raw_al = (raw + 1023u) & ~1023u;
                const unsigned int tb = parts * (unsigned int)(padded / 32) * 128u * (unsigned int)(g->m_chunk + tpc * n_cols);
                const unsigned int slack = g->m_chunk < 128 ? kWgradSlack : 0u;     // no over-read with 128 channel rows
                if (2 * raw_al + 2 * tb + slack > kWgradSmemBudget) continue;
                g->n_cols = n_cols;
                g->taps_per_cta = tpc;
                g->box = b; g->rows_padded = padded; g->raw_bytes = raw_al; g->t_bytes = tb;
                g->t_stages = 2;
                int rs = (int)((kWgradSmemBudget - slack - 2 * tb) / raw_al);
                g->raw_stages = rs > 2 ? 2 : rs;
                found = true;
            }
        }
    }
    if (!found) return false;
    g->tap_groups = (taps + g->taps_per_cta - 1) / g->taps_per_cta;
    g->tmem_cols = pow2_cols(g->taps_per_cta * g->n_cols);
    const int tiles_w = (s.Q + g->box.w - 1) / g->box.w, tiles_h = (s.P + g->box.h - 1) / g->box.h, tiles_n = (s.N + g->box.n - 1) / g->box.n;
    g->n_tiles = tiles_w * tiles_h * tiles_n;
    wgrad_splits(s, g->n_tiles, g->tap_groups * (s.K / g->m_chunk) * (s.C / g->n_cols), max_ctas, &g->splits, &g->tiles_per_split);
    return true;
}

struct WgradDirectGeom {
    PixelBox box;
    int m_chunk, n_cols, m_blocks, n_blocks, m_box, n_box, taps_per_cta, tap_groups, stages, splits, tiles_per_split, n_tiles, rows_padded;
    unsigned int stage_bytes, lo_off, slack, tmem_cols;
};

// Geometry of the kernel that reads its TMA tiles directly: output channels per CTA (up to 128), input channels per CTA
// (all up to 256, else 128 or 64), taps per CTA (all, one row of the window, or one) and pixels per tile (128, 64 or 32):
// the first combination whose accumulators take at most half of an SM's tensor memory (other kernels' CTAs share the
// SM) and that gets at least three pipeline stages into 100 KB of shared memory - failing that two stages, failing
// that two stages into 200 KB with all of the tensor memory.
bool wgrad_direct_geom(const ConvShape& s, int passes, WgradDirectGeom* g, int max_ctas = 0)
{
    if (s.C % 16 || s.K % 16) return false;
    if ((s.C > 16 && s.C % 32) || (s.K > 16 && s.K % 32)) return false;
    if (s.R != 1 && s.R != 3) return false;
    if (s.R == 3 && (s.stride != 1 || s.pad != 1)) return false;
    if (s.R == 1 && s.pad != 0) return false;
    if (s.stride < 1 || s.stride > 2) return false;
    // measured: nine taps of a 16-channel tensor, split into hi and lo, are faster through the transposing kernel (its
    // tiles of such a tensor are dense; here every pixel of it takes a 128-byte row)
    if (passes == 3 && s.R == 3 && (s.C == 16 || s.K == 16)) return false;
    g->m_chunk = s.K < 128 ? s.K : 128;
    if (s.K % g->m_chunk) return false;
    g->m_blocks = (g->m_chunk + 31) / 32;
    g->m_box = g->m_chunk < 32 ? g->m_chunk : 32;
    const int taps = s.R * s.R;
    const unsigned int parts = passes == 3 ? 2u : 1u;
    bool found = false;
    const int ncand[3] = {s.C < 256 ? s.C : 256, 128, 64};
    const int cand[3] = {taps, taps == 9 ? 3 : 1, 1};
    const unsigned int budgets[3] = {100u * 1024u, 100u * 1024u, 200u * 1024u};
    const unsigned int tmem_caps[3] = {256u, 256u, 512u};
    const int min_stages[3] = {3, 2, 2};
    for (int tier = 0; tier < 3 && !found; ++tier) {
        // three passes double every stage and put the hi / lo split on the four spare warps: two stages are then too few
        // to keep the tensor core fed, and the launch does better alone on an SM with long tiles
        if (tier == 1 && passes == 3) continue;
        for (int ni = 0; ni < 3 && !found; ++ni) {
            const int n_cols = ncand[ni];
            if (n_cols > s.C || s.C % n_cols || (ni > 0 && n_cols >= ncand[0])) continue;
            const int n_blocks = (n_cols + 31) / 32;
            for (int ci = 0; ci < 3 && !found; ++ci) {
                const int tpc = cand[ci];
                if (ci > 0 && tpc >= cand[0]) continue;
                if ((unsigned int)(tpc * n_blocks * 32) > tmem_caps[tier]) continue;
                for (int rows = 128; rows >= 32 && !found; rows >>= 1) {
                    PixelBox b;
                    if (!choose_box(s.Q, s.P, s.N, rows, 1, &b)) continue;
                    const int padded = (b.rows + 7) / 8 * 8;
                    const unsigned int half = (unsigned int)padded * 128u * (unsigned int)(g->m_blocks + tpc * n_blocks);
                    const unsigned int stage = parts * half;
                    // the dy operand is read as 4 blocks whatever it holds; in the last stage what follows the x tile is
                    // read too: room for that behind the last stage
                    const int stage_blocks = g->m_blocks + tpc * n_blocks;
                    const unsigned int slack = stage_blocks < 4 ? (unsigned int)(4 - stage_blocks) * (unsigned int)padded * 128u : 0u;
                    const int want_stages = min_stages[tier];
                    if ((unsigned int)want_stages * stage + slack > budgets[tier]) continue;
                    int st = (int)((budgets[tier] - slack) / stage);
                    if (st > 4) st = 4;
                    g->n_cols = n_cols; g->n_blocks = n_blocks; g->n_box = n_cols < 32 ? n_cols : 32;
                    g->taps_per_cta = tpc;
                    g->box = b; g->rows_padded = padded; g->stage_bytes = stage; g->lo_off = half; g->slack = slack; g->stages = st;
                    found = true;
                }
            }
        }
    }
    if (!found) return false;
    g->tap_groups = (taps + g->taps_per_cta - 1) / g->taps_per_cta;
    g->tmem_cols = pow2_cols(g->taps_per_cta * g->n_blocks * 32);
    const int tiles_w = (s.Q + g->box.w - 1) / g->box.w, tiles_h = (s.P + g->box.h - 1) / g->box.h, tiles_n = (s.N + g->box.n - 1) / g->box.n;
    g->n_tiles = tiles_w * tiles_h * tiles_n;
    wgrad_splits(s, g->n_tiles, g->tap_groups * (s.K / g->m_chunk) * (s.C / g->n_cols), max_ctas, &g->splits, &g->tiles_per_split);
    return true;
}

inline void count(int64_t* n_launch, int k) { if (n_launch) *n_launch += k; }

}  // namespace

// ------------------------------------------------------------------------------------------------
// interface
// ------------------------------------------------------------------------------------------------
bool conv_tc_supported(const ConvShape& s, int pass)
{
    if (pass == PASS_WGRAD) { WgradGeom g; return wgrad_geom(s, 3, &g); }
    FwdView v;
    if (!fwd_view(s, pass, &v)) return false;
    PixelBox b;
    return choose_box(v.Q, v.P, v.N, kTileM, 1, &b);
}

int conv_tc_tiles(const ConvShape& s, int pass)
{
    FwdView v;
    PixelBox b;
    if (pass == PASS_WGRAD || !fwd_view(s, pass, &v) || !choose_box(v.Q, v.P, v.N, kTileM, 1, &b)) return 0;
    return ((v.Q + b.w - 1) / b.w) * ((v.P + b.h - 1) / b.h) * ((v.N + b.n - 1) / b.n);
}

bool conv_tc_can_fuse_bn(const ConvShape& s, int pass)
{
    FwdView v;
    if (pass == PASS_WGRAD || !fwd_view(s, pass, &v)) return false;
    // the write-out keeps one group of 4 channels per thread and the last CTA combines 2*C columns with 256 threads:
    // a power of two between 16 and 256 channels, all in one channel slice
    const int C = v.c_out;
    if (!(C >= 16 && C <= 256 && (C & (C - 1)) == 0 && conv_tc_tiles(s, pass) > 0)) return false;
    // the per-tile moments are merged as equal-sized groups: every tile must be full
    PixelBox b;
    if (!choose_box(v.Q, v.P, v.N, kTileM, 1, &b)) return false;
    return v.Q % b.w == 0 && v.P % b.h == 0 && v.N % b.n == 0;
}

bool conv_tc_can_fuse_bn_input(const ConvShape& s)
{
    FwdView v;
    if (!fwd_view(s, PASS_FWD, &v) || s.stride != 1) return false;
    const int C = s.C;
    return C >= 16 && C <= 256 && (C & (C - 1)) == 0 && conv_tc_tiles(s, PASS_FWD) > 0;
}

cudaError_t conv_tc_init()
{
    if (g_encode) return cudaSuccess;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess) return e;
    if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    e = cudaFuncSetAttribute(conv_tc_fwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget + 2048);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(conv_tc_fwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget + 2048);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(conv_tc_fwd_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget + 2048);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(conv_tc_cell_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget + 2048);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(conv_tc_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWgradSmemBudget + 2048);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(conv_tc_wgrad_direct_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWgradSmemBudget + 2048);
    if (e != cudaSuccess) return e;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return cudaSuccess;
}

namespace {

// How many CTAs share one tile's K loop.  Launches of a few tiles whose K loop is long (512-channel 3x3 convolutions on 7x7 or
// 2x2 maps, fully connected layers) are bound by one CTA's MMA issue (about 0.1 us per K step of 8): splitting the loop
// shortens it, at the price of one partial tile per split kept in L2.
int splitk_factor(int tiles, int slices, int total_iters, int k8n)
{
    const int ctas = tiles * slices;
    if (ctas > 32) return 1;                     // more CTAs than that already spread over the GPU; splitting them cost more than it gave
    const int ksteps = total_iters * k8n;
    if (ksteps < 128) return 1;
    int S = 296 / ctas;
    if (S > 8) S = 8;
    if (S > ksteps / 32) S = ksteps / 32;        // at least 32 K steps per CTA
    if (S > total_iters) S = total_iters;
    return S < 2 ? 1 : S;
}

// Channel slice width of an unfused forward / data-gradient launch (see conv_tc_prepare).
int unfused_n_chunk(int c_out, int tiles)
{
    int n_chunk = c_out < 256 ? c_out : 256;
    if (c_out % 256 == 0 && tiles * (c_out / 256) <= 74) n_chunk = 128;
    return n_chunk;
}

}  // namespace

size_t conv_tc_splitk_bytes(const ConvShape& s, int pass, int passes)
{
    FwdView v;
    PixelBox b;
    if (pass == PASS_WGRAD || !fwd_view(s, pass, &v) || !choose_box(v.Q, v.P, v.N, kTileM, 1, &b)) return 0;
    (void)passes;
    const int tiles = ((v.Q + b.w - 1) / b.w) * ((v.P + b.h - 1) / b.h) * ((v.N + b.n - 1) / b.n);
    const int n_chunk = unfused_n_chunk(v.c_out, tiles);
    if (v.c_out % n_chunk) return 0;
    const int kchunk = chunk_of(v.c_in);
    const int S = splitk_factor(tiles, v.c_out / n_chunk, v.R * v.R * (v.c_in / kchunk), kchunk / 8);
    if (S < 2) return 0;
    return kSplitKTicketBytes + (size_t)tiles * (v.c_out / n_chunk) * S * kTileM * n_chunk * sizeof(float);
}

size_t conv_tc_scratch_bytes(const ConvShape& s)
{
    size_t need = 0;
    for (int passes = 1; passes <= 3; passes += 2) {
        WgradGeom g;
        if (!wgrad_geom(s, passes, &g)) continue;
        const size_t b = g.splits > 1 ? (size_t)g.splits * s.K * s.R * s.R * s.C * sizeof(float) : 0;
        if (b > need) need = b;
        WgradDirectGeom d;
        if (!wgrad_direct_geom(s, passes, &d)) continue;
        const size_t bd = d.splits > 1 ? (size_t)d.splits * s.K * s.R * s.R * s.C * sizeof(float) : 0;
        if (bd > need) need = bd;
    }
    return need;
}

struct ConvTcFwdLaunch { FwdParams p; dim3 grid; unsigned int smem; };
struct ConvTcWgradLaunch { WgradParams p; dim3 grid; unsigned int smem; int splits; float* dw; long long n_out; };
struct ConvTcWgradDirectLaunch { WgradDirectParams p; dim3 grid; unsigned int smem; int splits; float* dw; long long n_out; };
static_assert(sizeof(ConvTcWgradDirectLaunch) <= sizeof(((ConvTcPlan*)0)->storage), "plan storage too small");
static_assert(sizeof(ConvTcFwdLaunch) <= sizeof(((ConvTcPlan*)0)->storage) && sizeof(ConvTcWgradLaunch) <= sizeof(((ConvTcPlan*)0)->storage),
              "plan storage too small");

cudaError_t conv_tc_prepare(ConvTcPlan* plan, const ConvShape& s, int pass, int passes, const float* in, const float* in2,
                            const float* w_hi, const float* w_lo, float* out, const float* extra, bool accumulate, void* scratch,
                            const ConvBnFuse* fuse)
{
    plan->valid = 0; plan->s = s; plan->pass = pass; plan->direct = 0;
    if (passes != 1 && passes != 3) return cudaErrorInvalidValue;
    WgradDirectGeom dg;
    if (pass == PASS_WGRAD && !(fuse && fuse->wgrad_transposing) && wgrad_direct_geom(s, passes, &dg, fuse ? fuse->wgrad_max_ctas : 0)) {
        ConvTcWgradDirectLaunch* L = reinterpret_cast<ConvTcWgradDirectLaunch*>(plan->storage);
        WgradDirectParams& P = L->p;
        memset(&P, 0, sizeof P);
        WgradDirectScalars& p = P.s;
        {   // dy {K, Q, P, N}
            cuuint64_t dims[4] = {(cuuint64_t)s.K, (cuuint64_t)s.Q, (cuuint64_t)s.P, (cuuint64_t)s.N};
            cuuint64_t str[3] = {(cuuint64_t)s.K * 4, (cuuint64_t)s.Q * s.K * 4, (cuuint64_t)s.P * s.Q * s.K * 4};
            cuuint32_t box[4] = {(cuuint32_t)dg.m_box, (cuuint32_t)dg.box.w, (cuuint32_t)dg.box.h, (cuuint32_t)dg.box.n};
            cudaError_t e = encode(&P.tm_a, in, 4, dims, str, box, kSwizzle128Atom32);
            if (e != cudaSuccess) return e;
        }
        {   // x {C, Wv, Hv, N}: a strided 1x1 convolution samples every stride-th pixel
            const int wv = s.stride == 1 ? s.W : s.Q, hv = s.stride == 1 ? s.H : s.P;
            cuuint64_t dims[4] = {(cuuint64_t)s.C, (cuuint64_t)wv, (cuuint64_t)hv, (cuuint64_t)s.N};
            cuuint64_t str[3] = {(cuuint64_t)s.stride * s.C * 4, (cuuint64_t)s.stride * s.W * s.C * 4, (cuuint64_t)s.H * s.W * s.C * 4};
            cuuint32_t box[4] = {(cuuint32_t)dg.n_box, (cuuint32_t)dg.box.w, (cuuint32_t)dg.box.h, (cuuint32_t)dg.box.n};
            cudaError_t e = encode(&P.tm_b, in2, 4, dims, str, box, kSwizzle128Atom32);
            if (e != cudaSuccess) return e;
        }
        const long long n_out = (long long)s.K * s.R * s.R * s.C;
        p.out = dg.splits > 1 ? reinterpret_cast<float*>(scratch) : out;
        p.box_w = dg.box.w; p.box_h = dg.box.h; p.box_n = dg.box.n;
        p.tiles_w = (s.Q + dg.box.w - 1) / dg.box.w; p.tiles_h = (s.P + dg.box.h - 1) / dg.box.h;
        p.n_tiles = dg.n_tiles; p.tiles_per_split = dg.tiles_per_split; p.rows = dg.rows_padded; p.box_rows = dg.box.rows;
        p.c_out = s.K; p.c_in = s.C; p.R = s.R; p.pad = s.pad;
        p.m_chunk = dg.m_chunk; p.n_cols = dg.n_cols; p.m_blocks = dg.m_blocks; p.n_blocks = dg.n_blocks; p.m_box = dg.m_box; p.n_box = dg.n_box;
        p.taps_per_cta = dg.taps_per_cta; p.stages = dg.stages; p.passes = passes;
        p.stage_bytes = dg.stage_bytes; p.lo_off = dg.lo_off;
        p.tx_bytes_a = (unsigned int)dg.box.rows * dg.m_chunk * 4u; p.tx_per_tap = (unsigned int)dg.box.rows * dg.n_cols * 4u;
        p.tmem_cols = dg.tmem_cols;
        const int slot = dg.n_blocks * 32;
        p.taps_per_mma = 256 / slot < dg.taps_per_cta ? 256 / slot : dg.taps_per_cta;
        p.idesc = instr_desc(slot * p.taps_per_mma, true, true);
        p.idesc_tail = instr_desc(slot * (dg.taps_per_cta % p.taps_per_mma ? dg.taps_per_cta % p.taps_per_mma : p.taps_per_mma), true, true);
        p.split_stride = n_out;
        L->grid = dim3(dg.splits, dg.tap_groups, (s.K / dg.m_chunk) * (s.C / dg.n_cols));
        L->smem = (unsigned int)dg.stages * dg.stage_bytes + dg.slack + 1024;
        L->splits = dg.splits; L->dw = out; L->n_out = n_out;
        plan->direct = 1;
        plan->valid = 1;
        return cudaSuccess;
    }
    if (pass == PASS_WGRAD) {
        WgradGeom g;
        if (!wgrad_geom(s, passes, &g, fuse ? fuse->wgrad_max_ctas : 0)) return cudaErrorNotSupported;
        ConvTcWgradLaunch* L = reinterpret_cast<ConvTcWgradLaunch*>(plan->storage);
        WgradParams& P = L->p;
        memset(&P, 0, sizeof P);
        WgradScalars& p = P.s;
        // dy {K, Q, P, N}
        {
            cuuint64_t dims[4] = {(cuuint64_t)s.K, (cuuint64_t)s.Q, (cuuint64_t)s.P, (cuuint64_t)s.N};
            cuuint64_t str[3] = {(cuuint64_t)s.K * 4, (cuuint64_t)s.Q * s.K * 4, (cuuint64_t)s.P * s.Q * s.K * 4};
            cuuint32_t box[4] = {(cuuint32_t)g.m_chunk, (cuuint32_t)g.box.w, (cuuint32_t)g.box.h, (cuuint32_t)g.box.n};
            cudaError_t e = encode(&P.tm_a, in, 4, dims, str, box, 0);
            if (e != cudaSuccess) return e;
        }
        // x {C, Wv, Hv, N}: a strided 1x1 convolution samples every stride-th pixel
        {
            const int wv = s.stride == 1 ? s.W : s.Q, hv = s.stride == 1 ? s.H : s.P;
            cuuint64_t dims[4] = {(cuuint64_t)s.C, (cuuint64_t)wv, (cuuint64_t)hv, (cuuint64_t)s.N};
            cuuint64_t str[3] = {(cuuint64_t)s.stride * s.C * 4, (cuuint64_t)s.stride * s.W * s.C * 4, (cuuint64_t)s.H * s.W * s.C * 4};
            cuuint32_t box[4] = {(cuuint32_t)g.n_cols, (cuuint32_t)g.box.w, (cuuint32_t)g.box.h, (cuuint32_t)g.box.n};
            cudaError_t e = encode(&P.tm_b, in2, 4, dims, str, box, 0);
            if (e != cudaSuccess) return e;
        }
        const long long n_out = (long long)s.K * s.R * s.R * s.C;
        p.out = g.splits > 1 ? reinterpret_cast<float*>(scratch) : out;
        p.box_w = g.box.w; p.box_h = g.box.h; p.box_n = g.box.n;
        p.tiles_w = (s.Q + g.box.w - 1) / g.box.w; p.tiles_h = (s.P + g.box.h - 1) / g.box.h;
        p.n_tiles = g.n_tiles; p.tiles_per_split = g.tiles_per_split; p.rows = g.rows_padded; p.box_rows = g.box.rows;
        p.c_out = s.K; p.c_in = s.C; p.R = s.R; p.pad = s.pad;
        p.m_chunk = g.m_chunk; p.n_cols = g.n_cols; p.taps_per_cta = g.taps_per_cta;
        p.raw_stages = g.raw_stages; p.t_stages = g.t_stages; p.passes = passes;
        p.raw_bytes = g.raw_bytes; p.t_bytes = g.t_bytes;
        p.tx_a = (unsigned int)g.box.rows * g.m_chunk * 4u; p.tx_per_tap = (unsigned int)g.box.rows * g.n_cols * 4u;
        p.tmem_cols = g.tmem_cols;
        p.taps_per_mma = 256 / g.n_cols < g.taps_per_cta ? 256 / g.n_cols : g.taps_per_cta;
        p.idesc = instr_desc(g.n_cols * p.taps_per_mma, false, false);
        p.idesc_tail = instr_desc(g.n_cols * (g.taps_per_cta % p.taps_per_mma ? g.taps_per_cta % p.taps_per_mma : p.taps_per_mma), false, false);
        p.split_stride = n_out;
        L->grid = dim3(g.splits, g.tap_groups, (s.K / g.m_chunk) * (s.C / g.n_cols));
        L->smem = (unsigned int)g.raw_stages * g.raw_bytes + (unsigned int)g.t_stages * g.t_bytes + (g.m_chunk < 128 ? kWgradSlack : 0u) + 1024;
        L->splits = g.splits; L->dw = out; L->n_out = n_out;
        plan->valid = 1;
        return cudaSuccess;
    }
    FwdView v;
    PixelBox b;
    if (!fwd_view(s, pass, &v) || !choose_box(v.Q, v.P, v.N, kTileM, 1, &b)) return cudaErrorNotSupported;
    ConvTcFwdLaunch* L = reinterpret_cast<ConvTcFwdLaunch*>(plan->storage);
    FwdParams& P = L->p;
    memset(&P, 0, sizeof P);
    FwdScalars& p = P.s;
    const int kchunk = chunk_of(v.c_in);
    int n_chunk = v.c_out < 256 ? v.c_out : 256;
    {
        // A launch with few pixel tiles leaves most SMs idle: twice as many channel slices of 128 (two MMAs of the stacked
        // width per K step instead of three) fill them.  When BN work rides in the kernel every slice repeats the BN on its
        // copy of the activation tile, which only pays when the K loop is long (the wide convolutions of the ImageNet layout).
        const int tiles = ((v.Q + b.w - 1) / b.w) * ((v.P + b.h - 1) / b.h) * ((v.N + b.n - 1) / b.n);
        const bool fused = fuse && (fuse->mode || fuse->in_mode);
        const int ksteps = v.R * v.R * v.c_in / 8;
        if ((!fused || ksteps >= 64) && v.c_out % 256 == 0 && tiles * (v.c_out / 256) <= 74) n_chunk = 128;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)v.c_in, (cuuint64_t)v.in_w, (cuuint64_t)v.in_h, (cuuint64_t)v.N};
        cuuint64_t str[3] = {(cuuint64_t)v.in_sw * 4, (cuuint64_t)v.in_sh * 4, (cuuint64_t)v.in_sn * 4};
        cuuint32_t box[4] = {(cuuint32_t)kchunk, (cuuint32_t)b.w, (cuuint32_t)b.h, (cuuint32_t)b.n};
        cudaError_t e = encode(&P.tm_a, in, 4, dims, str, box, kchunk * 4);
        if (e != cudaSuccess) return e;
    }
    {
        const long long kdim = (long long)v.R * v.R * v.c_in;
        cuuint64_t dims[2] = {(cuuint64_t)kdim, (cuuint64_t)v.c_out};
        cuuint64_t str[1] = {(cuuint64_t)kdim * 4};
        cuuint32_t box[2] = {(cuuint32_t)kchunk, (cuuint32_t)n_chunk};
        cudaError_t e = encode(&P.tm_b, w_hi, 2, dims, str, box, kchunk * 4);
        if (e != cudaSuccess) return e;
        if (passes == 3) {
            e = encode(&P.tm_b_lo, w_lo, 2, dims, str, box, kchunk * 4);
            if (e != cudaSuccess) return e;
        }
    }
    if ((long long)v.N * v.os_n >= (1LL << 31)) return cudaErrorNotSupported;      // the write-out keeps 32-bit offsets
    p.out = out; p.extra = extra; p.accumulate = accumulate ? 1 : 0;
    p.os_n = v.os_n; p.os_h = v.os_h; p.os_w = v.os_w; p.dense_h = v.dense_h; p.dense_w = v.dense_w;
    p.box_w = b.w; p.box_h = b.h; p.box_n = b.n;
    p.tiles_w = (v.Q + b.w - 1) / b.w; p.tiles_h = (v.P + b.h - 1) / b.h;
    const int tiles_n = (v.N + b.n - 1) / b.n;
    p.P = v.P; p.Q = v.Q; p.N = v.N; p.c_out = v.c_out; p.n_chunk = n_chunk; p.R = v.R; p.pad = v.pad;
    p.c_in = v.c_in; p.kchunk = kchunk; p.n_kchunks = v.c_in / kchunk; p.swizzle = kchunk * 4;
    p.passes = passes;
    p.zero_fill = v.zero_fill; p.out_h = v.out_h; p.out_w = v.out_w;
    p.a_bytes = (unsigned int)kTileM * kchunk * 4;
    p.b_bytes = ((unsigned int)n_chunk * kchunk * 4 + 1023u) & ~1023u;
    const unsigned int parts = passes == 3 ? 2u : 1u;
    p.stage_bytes = parts * (p.a_bytes + p.b_bytes);
    p.tx_bytes = (unsigned int)b.rows * kchunk * 4 + parts * (unsigned int)n_chunk * kchunk * 4;
    int stages = (int)(kSmemBudget / p.stage_bytes);
    const int total = v.R * v.R * p.n_kchunks;
    if (stages > kFwdMaxStages) stages = kFwdMaxStages;      // measured: more stages cost more in residency than they hide
    // one more where two CTAs still fit an SM: nine taps then take two rounds of the ring instead of three
    if (total > kFwdMaxStages && (unsigned int)(kFwdMaxStages + 1) * p.stage_bytes <= 92u * 1024u) stages = kFwdMaxStages + 1;
    if (stages > total) stages = total;
    const int cell_ctas = fuse ? fuse->cell_ctas : 0;
    const unsigned int cell_budget = cell_ctas > 0 ? (fuse->cell_smem ? fuse->cell_smem : kCellSmemBudget) : 0u;
    if (cell_ctas > 0)
        while (stages > 1 && (unsigned int)stages * p.stage_bytes > cell_budget) --stages;
    p.stages = stages;
    if (fuse && fuse->mode) {
        if (256 % (n_chunk / 4)) return cudaErrorNotSupported;
        if ((fuse->mode != 1 && fuse->mode != 3) || pass != PASS_FWD || !conv_tc_can_fuse_bn(s, pass) || fuse->rows < 1) return cudaErrorNotSupported;
        p.stat_mode = fuse->mode; p.stat_partials = fuse->partials;
        p.stat_ticket = fuse->ticket; p.stat_out = fuse->stats_out; p.stat_eps = fuse->eps; p.stat_inv_rows = 1.0 / (double)fuse->rows;
        p.stat_inv_tile_rows = 1.0f / (float)b.rows;
    }
    if (fuse && fuse->in_mode) {
        if (pass != PASS_FWD || !conv_tc_can_fuse_bn_input(s)) return cudaErrorNotSupported;
        if (fuse->in_mode != 1 && fuse->in_mode != 2) return cudaErrorInvalidValue;
        if (fuse->in_mode == 2 && (fuse->in_tiles < 1 || fuse->in_rows < 1 || !fuse->in_partials)) return cudaErrorInvalidValue;
        p.bn_in = fuse->in_mode; p.in_w = v.in_w; p.in_h = v.in_h;
        p.bn_in_gamma = fuse->in_gamma; p.bn_in_beta = fuse->in_beta;
        p.bn_in_stats = fuse->in_stats; p.bn_in_y = fuse->in_y;
        p.bn_in_partials = fuse->in_partials; p.bn_in_stats_out = fuse->in_stats; p.bn_in_tiles = fuse->in_tiles;
        p.bn_in_eps = fuse->in_eps; p.bn_in_inv_rows = fuse->in_rows > 0 ? 1.0 / (double)fuse->in_rows : 0.0;
    }
    p.stacked = (passes == 3 && 2 * n_chunk <= 256) ? 1 : 0;
    p.acc_cols = (unsigned int)(p.stacked ? 2 * n_chunk : n_chunk);
    p.idesc = instr_desc(n_chunk, false, false);
    p.idesc2 = instr_desc(p.stacked ? 2 * n_chunk : n_chunk, false, false);
    p.stg_pitch = (unsigned int)n_chunk + 4u;
    p.n_tiles = p.tiles_w * p.tiles_h * tiles_n;
    const unsigned int pipe_bytes = (unsigned int)stages * p.stage_bytes;
    const unsigned int stg_bytes = (unsigned int)kTileM * p.stg_pitch * 4u;
    // Two tiles per CTA when the launch is several waves long anyway: half as many CTAs, and the second tile's loads and
    // MMAs hide under the first tile's write-out.  Needs twice the accumulator columns (two such CTAs must still fit
    // the 512 columns of an SM) and a staging area beside the pipeline.  A launch of about a wave keeps one tile per
    // CTA: there the duration of the launch is one CTA's own chain.
    p.tiles_per_cta = 1;
    if (cell_ctas > 0) {
        // inside a persistent cell kernel of cell_ctas CTAs: as many tiles per CTA as bring the launch down to one round of
        // the grid, within four accumulator barriers, the cell's tensor-memory columns and its shared memory
        int t = (p.n_tiles * (v.c_out / n_chunk) + cell_ctas - 1) / cell_ctas;
        if (t > 4) t = 4;
        while (t > 1 && (unsigned int)t * p.acc_cols > kCellTmemCols) --t;
        if (t > 1 && pipe_bytes + stg_bytes > cell_budget) t = 1;
        p.tiles_per_cta = t < 1 ? 1 : t;
    } else if (p.n_tiles * (v.c_out / n_chunk) >= kMultiTileFrom && 2 * p.acc_cols <= 256 && pipe_bytes + stg_bytes <= 110u * 1024u) {
        int t = (p.n_tiles * (v.c_out / n_chunk) + 295) / 296;            // tiles per CTA that bring the launch down to one wave
        if (t > 4) t = 4;                                                 // accumulator barriers
        while (t > 2 && (unsigned int)t * p.acc_cols > 256u) --t;
        p.tiles_per_cta = t < 2 ? 2 : t;
    }
    p.pdl_late = fuse && fuse->pdl_late ? 1 : 0;
    p.ksplit = 1;
    if (fuse && fuse->splitk && !fuse->mode && !fuse->in_mode && p.tiles_per_cta == 1) {
        const int S = splitk_factor(p.n_tiles, v.c_out / n_chunk, total, kchunk / 8);
        const size_t need = kSplitKTicketBytes + (size_t)p.n_tiles * (v.c_out / n_chunk) * S * kTileM * n_chunk * sizeof(float);
        if (S > 1 && need <= fuse->splitk_bytes) {
            p.ksplit = S;
            p.splitk_ticket = reinterpret_cast<unsigned int*>(fuse->splitk);
            p.splitk_partials = reinterpret_cast<float*>(reinterpret_cast<char*>(fuse->splitk) + kSplitKTicketBytes);
            const int per_cta = total / S;                   // the shortest share of the K loop
            if (p.stages > per_cta) p.stages = per_cta < 1 ? 1 : per_cta;
        }
    }
    p.tmem_cols = pow2_cols((int)p.acc_cols * p.tiles_per_cta);
    p.stg_off = p.tiles_per_cta > 1 ? pipe_bytes : 0u;
    L->grid = dim3((p.n_tiles + p.tiles_per_cta - 1) / p.tiles_per_cta, v.c_out / n_chunk, p.ksplit);
    L->smem = p.tiles_per_cta > 1 ? pipe_bytes + stg_bytes : (pipe_bytes > stg_bytes ? pipe_bytes : stg_bytes);
    L->smem += 1024;
    if (p.stat_mode == 1 && L->smem < 8192u + 1024u) L->smem = 8192u + 1024u;      // the last CTA's reduction: 8 x 32 x 8 floats
    plan->valid = 1;
    return cudaSuccess;
}

cudaError_t conv_tc_launch(const ConvTcPlan* plan, DeviceStatus* status, cudaStream_t st, int64_t* n_launch)
{
    if (!plan->valid) return cudaErrorInvalidValue;
    if (plan->pass == PASS_WGRAD && plan->direct) {
        ConvTcWgradDirectLaunch L = *reinterpret_cast<const ConvTcWgradDirectLaunch*>(plan->storage);
        L.p.s.status = status;
        launch_pdl(conv_tc_wgrad_direct_kernel, L.grid, dim3(192), L.smem, st, L.p);
        count(n_launch, 1);
        if (L.splits > 1) {
            const int nb = (int)((L.n_out / 4 + 31) / 32);
            launch_pdl(wgrad_partials_reduce_kernel, dim3(nb), dim3(256), 0, st, (const float*)L.p.s.out, L.dw, L.n_out, L.splits);
            count(n_launch, 1);
        }
        return cudaGetLastError();
    }
    if (plan->pass == PASS_WGRAD) {
        ConvTcWgradLaunch L = *reinterpret_cast<const ConvTcWgradLaunch*>(plan->storage);
        L.p.s.status = status;
        launch_pdl(conv_tc_wgrad_kernel, L.grid, dim3(192), L.smem, st, L.p);
        count(n_launch, 1);
        if (L.splits > 1) {
            const int nb = (int)((L.n_out / 4 + 31) / 32);
            launch_pdl(wgrad_partials_reduce_kernel, dim3(nb), dim3(256), 0, st, (const float*)L.p.s.out, L.dw, L.n_out, L.splits);
            count(n_launch, 1);
        }
        return cudaGetLastError();
    }
    ConvTcFwdLaunch L = *reinterpret_cast<const ConvTcFwdLaunch*>(plan->storage);
    L.p.s.status = status;
    if (L.p.s.ksplit > 1) launch_pdl(conv_tc_fwd_kernel<false, true>, L.grid, dim3(320), L.smem, st, L.p);
    else if (L.p.s.tiles_per_cta > 1) launch_pdl(conv_tc_fwd_kernel<true>, L.grid, dim3(320), L.smem, st, L.p);
    else launch_pdl(conv_tc_fwd_kernel<false>, L.grid, dim3(320), L.smem, st, L.p);
    count(n_launch, 1);
    return cudaGetLastError();
}

size_t conv_tc_cell_op_bytes() { return sizeof(CellOp); }

cudaError_t conv_tc_cell_op(const ConvTcPlan* plan, DeviceStatus* status, void* dst_host, unsigned int* smem, unsigned int* tmem_cols,
                            unsigned int* ctas)
{
    if (!plan->valid || plan->pass == PASS_WGRAD) return cudaErrorInvalidValue;
    const ConvTcFwdLaunch* L = reinterpret_cast<const ConvTcFwdLaunch*>(plan->storage);
    CellOp op;
    memset(&op, 0, sizeof op);
    op.p = L->p;
    op.p.s.status = status;
    op.gx = L->grid.x; op.gy = L->grid.y; op.gz = L->grid.z;
    memcpy(dst_host, &op, sizeof op);
    if (L->p.s.tmem_cols > kCellTmemCols) return cudaErrorNotSupported;
    *smem = L->smem; *tmem_cols = L->p.s.tmem_cols; *ctas = L->grid.x * L->grid.y * L->grid.z;
    return cudaSuccess;
}

void conv_tc_plan_pipeline(const ConvTcPlan* plan, int* stages, int* k_iterations)
{
    const ConvTcFwdLaunch* L = reinterpret_cast<const ConvTcFwdLaunch*>(plan->storage);
    *stages = L->p.s.stages; *k_iterations = L->p.s.R * L->p.s.R * L->p.s.n_kchunks;
}

int conv_tc_cell_max_ctas(unsigned int smem)
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, conv_tc_cell_kernel, 320, smem) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    if (per_sm > 2) per_sm = 2;          // two cell CTAs hold an SM's 512 tensor-memory columns between them
    return per_sm * sms;
}

cudaError_t conv_tc_cell_launch(const void* d_ops, int n_ops, int ctas, unsigned int smem, unsigned int tmem_cols, unsigned int* d_barrier,
                                DeviceStatus* status, cudaStream_t st, int64_t* n_launch)
{
    if (n_ops < 1 || ctas < 1 || tmem_cols < 32 || tmem_cols > kCellTmemCols) return cudaErrorInvalidValue;
    CellParams cp;
    cp.ops = reinterpret_cast<const CellOp*>(d_ops); cp.n_ops = n_ops; cp.barrier = d_barrier; cp.status = status; cp.tmem_cols = tmem_cols;
    // a plain stream-ordered launch: a resident grid that started early would only hold SM slots while it waits
    conv_tc_cell_kernel<<<dim3(ctas), dim3(320), smem, st>>>(cp);
    count(n_launch, 1);
    return cudaGetLastError();
}

int conv_weight_prep_tiles(int C, int K, int R) { return R * R * ((C + 31) / 32) * ((K + 31) / 32); }

cudaError_t conv_weight_prep(const float* params, float* w_hi, float* w_lo, float* wt_hi, float* wt_lo,
                             const WeightPrepEntry* d_table, int n_entries, int max_tiles, cudaStream_t st, int64_t* n_launch)
{
    if (n_entries < 1) return cudaSuccess;
    int gy = max_tiles < 1 ? 1 : max_tiles;                  // tiles of the largest entry; smaller entries leave blocks idle
    const int cap = n_entries >= 16 ? 64 : 2048;
    if (gy > cap) gy = cap;
    weight_prep_kernel<<<dim3(n_entries, gy), 256, 0, st>>>(params, w_hi, w_lo, wt_hi, wt_lo, d_table);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t conv_weight_prep_single(const float* w, float* w_hi, float* w_lo, float* wt_hi, float* wt_lo, int C, int K, int R,
                                    cudaStream_t st, int64_t* n_launch)
{
    WeightPrepEntry e{0, C, K, R, 0};
    int gy = conv_weight_prep_tiles(C, K, R);
    if (gy > 2048) gy = 2048;
    weight_prep_single_kernel<<<dim3(1, gy), 256, 0, st>>>(w, w_hi, w_lo, wt_hi, wt_lo, e);
    count(n_launch, 1);
    return cudaGetLastError();
}

}  // namespace hpf

#if defined(HPF_TC_TIMELINE) && HPF_TC_TIMELINE == 2
extern "C" int hpf_debug_timeline(unsigned long long* h_out, int reset)
{
    cudaDeviceSynchronize();
    if (h_out && cudaMemcpyFromSymbol(h_out, hpf::g_tl_acc, sizeof(unsigned long long) * 8 * 16) != cudaSuccess) return -1;
    if (reset) {
        static unsigned long long zeros[8 * 16];
        if (cudaMemcpyToSymbol(hpf::g_tl_acc, zeros, sizeof zeros) != cudaSuccess) return -1;
    }
    return 0;
}
#endif
