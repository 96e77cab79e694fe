// Memory-bound kernels of the step: fused BN(training)+ReLU forward/backward, residual add,
// gradient accumulate/average, max-pool and the pool+FC+softmax-CE head.  sm_100a.
//
// All tensors are fp32 with channels innermost.  Loads and stores are 128-bit and coalesced:
// consecutive threads walk consecutive float4 of a row-major [rows][C] tensor.
#include "hpf_kernels.h"

#include <cooperative_groups.h>
#include <math.h>

namespace hpf {

thread_local bool g_pdl_enabled = true;
thread_local bool g_bn_cluster = true;

namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 148 * 4;

__host__ __device__ inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------------------------------------
// BN + ReLU.  z = gamma * ((x - mean) * rstd) + beta, y = max(z, floor).  The same expression is used by
// the forward and by the backward mask (z > floor), so both take the ReLU decision on identical fp32 values.
// floor = 0 is BN+ReLU; floor = -infinity is batch normalisation without the activation (every element passes).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float bn_xhat(float x, float mean, float rstd) { return (x - mean) * rstd; }
__device__ __forceinline__ float bn_z(float xh, float g, float b) { return fmaf(g, xh, b); }

// Thread layout shared by the BN kernels: a block of kBnThreads threads is (row lanes) x (float4 column groups);
// a thread keeps its column group for the whole kernel, so per-channel coefficients live in registers and no
// index arithmetic runs per element.
constexpr int kBnThreads = 512;
constexpr int kBnMaxBlocks = 128;        // bounds the partials the last block has to combine (micro-batch sized tensors)
constexpr int kBnMaxBlocksLarge = 296;   // tensors beyond L2-resident sizes need more loads in flight: two blocks per SM
constexpr int64_t kBnLargeElems = 2 << 20;

struct BnPlan {
    int cg_total;        // float4 column groups = C/4
    int cgt;             // column groups handled per pass by one block (<= kBnThreads)
    int rl;              // row lanes per block = kBnThreads / cgt
    int passes;          // ceil(cg_total / cgt)
    int nblk;            // blocks of the reduction kernels
    int64_t rows_per_blk;
    int nblk_apply;      // blocks of the apply kernels (no partials: as many as the rows allow)
    int64_t rows_per_blk_apply;
};

BnPlan bn_plan(int64_t rows, int C)
{
    BnPlan p;
    p.cg_total = C / 4;
    p.cgt = p.cg_total < kBnThreads ? p.cg_total : kBnThreads;
    p.rl = kBnThreads / p.cgt;
    p.passes = (p.cg_total + p.cgt - 1) / p.cgt;
    // Four rows per thread (one batch of loads in flight, one memory round trip) while that keeps the partials few;
    // eight beyond, where the last block's combine and the ticket traffic would outweigh the shorter row loop.
    int64_t nb = rows / ((int64_t)p.rl * 4);
    if (nb > kBnMaxBlocks) nb = rows / ((int64_t)p.rl * 8) > kBnMaxBlocks ? rows / ((int64_t)p.rl * 8) : kBnMaxBlocks;
    if (nb < 1) nb = 1;
    const int cap = rows * C > kBnLargeElems ? kBnMaxBlocksLarge : kBnMaxBlocks;
    if (nb > cap) nb = cap;
    p.rows_per_blk = ceil_div64(rows, nb);
    p.nblk = (int)ceil_div64(rows, p.rows_per_blk);
    int64_t na = rows / ((int64_t)p.rl * 4);
    if (na < 1) na = 1;
    if (na > 148 * 8) na = 148 * 8;
    p.rows_per_blk_apply = ceil_div64(rows, na);
    p.nblk_apply = (int)ceil_div64(rows, p.rows_per_blk_apply);
    return p;
}

// Per-channel reductions over the rows.
//   forward  (BWD = false): a = sum (x - shift), b = sum (x - shift)^2 with shift = x[row 0][c]
//                           -> mean, rstd = 1/sqrt(var + eps)      (shifted sums avoid cancellation)
//   backward (BWD = true):  a = sum dz, b = sum dz * xhat, dz = dy * [z > 0]
//                           -> dbeta, dgamma and the two per-row coefficients of the dx formula
// Each block reduces its slab of rows and writes one partial per channel; the block that takes the last
// ticket combines the partials: every thread adds a fixed subset in ascending block order (fp64), a fixed
// tree adds those, so the result does not depend on which block happens to finish last.
template <bool BWD>
__global__ void __launch_bounds__(kBnThreads)
bn_reduce_kernel(const float* __restrict__ x, const float* __restrict__ dy, const float* __restrict__ gamma,
                 const float* __restrict__ beta, const float* __restrict__ stats, float eps, int64_t rows, int C,
                 int cgt, int rl, int passes, int64_t rows_per_blk, unsigned int* ticket,
                 float* __restrict__ partials, float* __restrict__ out_a, float* __restrict__ out_b,
                 float* __restrict__ coef, float floor)
{
    __shared__ double shd[kBnThreads][8];            // 32 KB; the float phase uses it as float[kBnThreads][8]
    float (*sh)[8] = reinterpret_cast<float (*)[8]>(&shd[0][0]);
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int is_last;
    const int t = threadIdx.x;
    const int cg_total = C / 4;
    const int my_rl = t / cgt, my_cg = t % cgt;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_blk;
    int64_t r1 = r0 + rows_per_blk;
    if (r1 > rows) r1 = rows;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const float4* dy4 = reinterpret_cast<const float4*>(dy);
    // all column groups in one pass, a power-of-two count of at most 16: the reductions over row lanes use warp shuffles
    const bool narrow = passes == 1 && cgt == cg_total && cgt <= 16 && (cgt & (cgt - 1)) == 0 && cgt * rl == kBnThreads;

    for (int pass = 0; pass < passes; ++pass) {
        const int cg = pass * cgt + my_cg;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (my_rl < rl && cg < cg_total) {
            float4 p0, p1, gm, bt;
            if (BWD) {
                p0 = __ldg(reinterpret_cast<const float4*>(stats) + cg);              // mean
                p1 = __ldg(reinterpret_cast<const float4*>(stats + C) + cg);          // rstd
                gm = __ldg(reinterpret_cast<const float4*>(gamma) + cg);
                bt = __ldg(reinterpret_cast<const float4*>(beta) + cg);
            } else {
                p0 = __ldg(x4 + cg);                                                  // shift = first row
            }
            const float4* xp = x4 + (r0 + my_rl) * cg_total + cg;
            const float4* dp = dy4 + (r0 + my_rl) * cg_total + cg;
            const int64_t step = (int64_t)rl * cg_total;
            const int n = (int)((r1 - r0 - my_rl + rl - 1) / rl);
#pragma unroll 4
            for (int k = 0; k < n; ++k) {
                const float4 v = __ldg(xp + k * step);
                if (BWD) {
                    const float4 g = __ldg(dp + k * step);
                    float xh, dz;
                    xh = bn_xhat(v.x, p0.x, p1.x); dz = bn_z(xh, gm.x, bt.x) > floor ? g.x : 0.f; a.x += dz; b.x = fmaf(dz, xh, b.x);
                    xh = bn_xhat(v.y, p0.y, p1.y); dz = bn_z(xh, gm.y, bt.y) > floor ? g.y : 0.f; a.y += dz; b.y = fmaf(dz, xh, b.y);
                    xh = bn_xhat(v.z, p0.z, p1.z); dz = bn_z(xh, gm.z, bt.z) > floor ? g.z : 0.f; a.z += dz; b.z = fmaf(dz, xh, b.z);
                    xh = bn_xhat(v.w, p0.w, p1.w); dz = bn_z(xh, gm.w, bt.w) > floor ? g.w : 0.f; a.w += dz; b.w = fmaf(dz, xh, b.w);
                } else {
                    float d;
                    d = v.x - p0.x; a.x += d; b.x = fmaf(d, d, b.x);
                    d = v.y - p0.y; a.y += d; b.y = fmaf(d, d, b.y);
                    d = v.z - p0.z; a.z += d; b.z = fmaf(d, d, b.z);
                    d = v.w - p0.w; a.w += d; b.w = fmaf(d, d, b.w);
                }
            }
        }
        if (narrow) {
            // Few column groups (cgt a power of two <= 16, so 32 / cgt row lanes of a group sit in one warp): a fixed
            // butterfly over the warp's row lanes, then the 16 warps' totals are added in ascending order.
            for (int off = 16; off >= cgt; off >>= 1) {
                a.x += __shfl_xor_sync(0xffffffffu, a.x, off); a.y += __shfl_xor_sync(0xffffffffu, a.y, off);
                a.z += __shfl_xor_sync(0xffffffffu, a.z, off); a.w += __shfl_xor_sync(0xffffffffu, a.w, off);
                b.x += __shfl_xor_sync(0xffffffffu, b.x, off); b.y += __shfl_xor_sync(0xffffffffu, b.y, off);
                b.z += __shfl_xor_sync(0xffffffffu, b.z, off); b.w += __shfl_xor_sync(0xffffffffu, b.w, off);
            }
            const int warp = t >> 5, lane = t & 31;
            if (lane < cgt) {
                float* d = sh[warp * cgt + lane];
                d[0] = a.x; d[1] = a.y; d[2] = a.z; d[3] = a.w; d[4] = b.x; d[5] = b.y; d[6] = b.z; d[7] = b.w;
            }
            __syncthreads();
            if (t < cgt * 8) {
                const int cgl = t >> 3, comp = t & 7;
                if (cgl < cg_total) {
                    float s = 0.f;
                    for (int w = 0; w < kBnThreads / 32; ++w) s += sh[w * cgt + cgl][comp];
                    partials[((int64_t)blockIdx.x * 2 + (comp >> 2)) * C + cgl * 4 + (comp & 3)] = s;
                }
            }
            __syncthreads();
            continue;
        }
        sh[t][0] = a.x; sh[t][1] = a.y; sh[t][2] = a.z; sh[t][3] = a.w;
        sh[t][4] = b.x; sh[t][5] = b.y; sh[t][6] = b.z; sh[t][7] = b.w;
        __syncthreads();
        // one output per (column group, component): add the row lanes in ascending order
        for (int o = t; o < cgt * 8; o += kBnThreads) {
            const int cgl = o >> 3, comp = o & 7;
            const int cgo = pass * cgt + cgl;
            if (cgo < cg_total) {
                float s = 0.f;
                for (int l = 0; l < rl; ++l) s += sh[l * cgt + cgl][comp];
                const int c = cgo * 4 + (comp & 3);
                partials[((int64_t)blockIdx.x * 2 + (comp >> 2)) * C + c] = s;
            }
        }
        __syncthreads();
    }

    __threadfence();
    __syncthreads();
    if (t == 0) {
        const unsigned int old = atomicAdd(ticket, 1u);
        is_last = (old == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // combine: thread (lane l, column group) adds the partials of blocks l, l+rl, ... (both sums, 4 channels each)
    const double inv_rows = 1.0 / (double)rows;
    const int nb = (int)gridDim.x;
    for (int pass = 0; pass < passes; ++pass) {
        const int cg = pass * cgt + my_cg;
        double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
        if (my_rl < rl && cg < cg_total) {
            // four partial rows per batch, their eight loads in flight together
            for (int k0 = my_rl; k0 < nb; k0 += 4 * rl) {
                float4 va[4], vb[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int k = k0 + j * rl;
                    const bool in = k < nb;
                    va[j] = in ? __ldcg(reinterpret_cast<const float4*>(partials + ((int64_t)k * 2 + 0) * C) + cg) : make_float4(0.f, 0.f, 0.f, 0.f);
                    vb[j] = in ? __ldcg(reinterpret_cast<const float4*>(partials + ((int64_t)k * 2 + 1) * C) + cg) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[0] += (double)va[j].x; acc[1] += (double)va[j].y; acc[2] += (double)va[j].z; acc[3] += (double)va[j].w;
                    acc[4] += (double)vb[j].x; acc[5] += (double)vb[j].y; acc[6] += (double)vb[j].z; acc[7] += (double)vb[j].w;
                }
            }
        }
        __syncthreads();
        if (narrow) {
            for (int off = 16; off >= cgt; off >>= 1) {
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], off);
            }
            const int warp = t >> 5, lane = t & 31;
            double (*wsum)[8] = shd + kBnThreads / 2;       // upper half of the buffer: [warp * cgt + column group][8]
            if (lane < cgt) {
#pragma unroll
                for (int j = 0; j < 8; ++j) wsum[warp * cgt + lane][j] = acc[j];
            }
            __syncthreads();
            if (t < cgt * 8) {
                const int cgl = t >> 3, comp = t & 7;
                double s = 0.0;
                for (int w = 0; w < kBnThreads / 32; ++w) s += wsum[w * cgt + cgl][comp];
                shd[cgl][comp] = s;                         // lower half: the totals, read below
            }
        } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) shd[t][j] = acc[j];
        __syncthreads();
        for (int o = t; o < cgt * 8; o += kBnThreads) {
            const int cgl = o >> 3, comp = o & 7;
            const int cgo = pass * cgt + cgl;
            if (cgo >= cg_total) continue;
            double s = 0.0;
            for (int l = 0; l < rl; ++l) s += shd[l * cgt + cgl][comp];
            // the pair (a, b) of one channel is finished by two threads: exchange through shared memory
            shd[cgl][comp] = s;       // row 0 lane (l = 0) slot of this column group: safe, every read above is done per o
        }
        }
        __syncthreads();
        for (int cl = t; cl < cgt * 4; cl += kBnThreads) {
            const int cgl = cl >> 2, e = cl & 3;
            const int cgo = pass * cgt + cgl;
            if (cgo >= cg_total) continue;
            const int c = cgo * 4 + e;
            const double sa = shd[cgl][e], sb = shd[cgl][4 + e];
            if (BWD) {
                out_a[c] = (float)sa;                 // dbeta
                out_b[c] = (float)sb;                 // dgamma
                coef[c] = (float)(sa * inv_rows);
                coef[C + c] = (float)(sb * inv_rows);
            } else {
                const double shift = (double)__ldg(x + c);
                const double ms = sa * inv_rows;
                double var = sb * inv_rows - ms * ms;
                if (var < 0.0) var = 0.0;
                out_a[c] = (float)(shift + ms);                       // mean
                out_b[c] = (float)(1.0 / sqrt(var + (double)eps));    // rstd
            }
        }
        __syncthreads();
    }
    if (t == 0) *ticket = 0u;
}

__global__ void __launch_bounds__(kBnThreads)
bn_apply_fwd_kernel(const float4* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                    const float* __restrict__ stats, float4* __restrict__ y, int64_t rows, int C, int cgt, int rl,
                    int passes, int64_t rows_per_blk, float floor)
{
    pdl_launch_dependents();
    pdl_wait();
    const int t = threadIdx.x, cg_total = C / 4;
    const int my_rl = t / cgt, my_cg = t % cgt;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_blk;
    int64_t r1 = r0 + rows_per_blk;
    if (r1 > rows) r1 = rows;
    if (my_rl >= rl) return;
    for (int pass = 0; pass < passes; ++pass) {
        const int cg = pass * cgt + my_cg;
        if (cg >= cg_total) continue;
        const float4 mu = __ldg(reinterpret_cast<const float4*>(stats) + cg);
        const float4 rs = __ldg(reinterpret_cast<const float4*>(stats + C) + cg);
        const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + cg);
        const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + cg);
        const int64_t base = (r0 + my_rl) * cg_total + cg, step = (int64_t)rl * cg_total;
        const int n = (int)((r1 - r0 - my_rl + rl - 1) / rl);
#pragma unroll 4
        for (int k = 0; k < n; ++k) {
            const float4 v = __ldg(x + base + k * step);
            float4 o;
            o.x = fmaxf(bn_z(bn_xhat(v.x, mu.x, rs.x), g.x, b.x), floor);
            o.y = fmaxf(bn_z(bn_xhat(v.y, mu.y, rs.y), g.y, b.y), floor);
            o.z = fmaxf(bn_z(bn_xhat(v.z, mu.z, rs.z), g.z, b.z), floor);
            o.w = fmaxf(bn_z(bn_xhat(v.w, mu.w, rs.w), g.w, b.w), floor);
            y[base + k * step] = o;
        }
    }
}

__device__ __forceinline__ float bn_dx1(float x, float dy, float mu, float rs, float g, float b, float ca, float cb, float floor)
{
    const float xh = bn_xhat(x, mu, rs);
    const float dz = bn_z(xh, g, b) > floor ? dy : 0.f;
    return g * rs * (dz - ca - xh * cb);
}

template <bool ADDEND, bool ACCUM>
__global__ void __launch_bounds__(kBnThreads)
bn_apply_bwd_kernel(const float4* __restrict__ x, const float4* __restrict__ dy, const float* __restrict__ gamma,
                    const float* __restrict__ beta, const float* __restrict__ stats, const float* __restrict__ coef,
                    const float4* __restrict__ addend, float4* __restrict__ dx, int64_t rows, int C, int cgt, int rl,
                    int passes, int64_t rows_per_blk, float floor)
{
    pdl_launch_dependents();
    pdl_wait();
    const int t = threadIdx.x, cg_total = C / 4;
    const int my_rl = t / cgt, my_cg = t % cgt;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_blk;
    int64_t r1 = r0 + rows_per_blk;
    if (r1 > rows) r1 = rows;
    if (my_rl >= rl) return;
    for (int pass = 0; pass < passes; ++pass) {
        const int cg = pass * cgt + my_cg;
        if (cg >= cg_total) continue;
        const float4 mu = __ldg(reinterpret_cast<const float4*>(stats) + cg);
        const float4 rs = __ldg(reinterpret_cast<const float4*>(stats + C) + cg);
        const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + cg);
        const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + cg);
        const float4 ca = __ldcg(reinterpret_cast<const float4*>(coef) + cg);
        const float4 cb = __ldcg(reinterpret_cast<const float4*>(coef + C) + cg);
        const int64_t base = (r0 + my_rl) * cg_total + cg, step = (int64_t)rl * cg_total;
        const int n = (int)((r1 - r0 - my_rl + rl - 1) / rl);
#pragma unroll 4
        for (int k = 0; k < n; ++k) {
            const int64_t i = base + k * step;
            const float4 v = __ldg(x + i);
            const float4 d = __ldg(dy + i);
            float4 o;
            o.x = bn_dx1(v.x, d.x, mu.x, rs.x, g.x, b.x, ca.x, cb.x, floor);
            o.y = bn_dx1(v.y, d.y, mu.y, rs.y, g.y, b.y, ca.y, cb.y, floor);
            o.z = bn_dx1(v.z, d.z, mu.z, rs.z, g.z, b.z, ca.z, cb.z, floor);
            o.w = bn_dx1(v.w, d.w, mu.w, rs.w, g.w, b.w, ca.w, cb.w, floor);
            if (ADDEND) { const float4 e = __ldg(addend + i); o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            if (ACCUM) { const float4 e = dx[i]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            dx[i] = o;
        }
    }
}

// BN(+ReLU) backward of a micro-batch sized tensor in ONE launch: thread-block clusters instead of the reduce / apply pair.
// A cluster of kBnCluster CTAs owns cgc float4 column groups (channels never mix, so clusters are independent); its CTAs
// split the rows.  Every thread keeps its NV rows of x and dy in registers, the CTA reduces sum dz and sum dz*xhat per
// channel (warp butterfly over the row lanes, then the warps in ascending order), the cluster's CTAs read each other's
// per-channel sums through distributed shared memory in ascending rank order (fp64), and dx is computed from the registers:
// one trip to memory for the operands, no partials in global memory, no ticket, no second kernel.
// early_x: x, the statistics and the BN parameters are not produced by the kernels just before this one (they are forward
// results), so they are fetched before the wait on the preceding kernel and only dy after it.
constexpr int kBnCluster = 8;
constexpr int kBnClusterMaxCgc = 16;
constexpr int kBnClusterMaxActive = 14;   // clusters of 8 one-per-SM CTAs that are resident together (15 measured); more would run as a second wave

template <int NV, bool ADDEND, bool ACCUM>
__global__ void __launch_bounds__(kBnThreads)
bn_bwd_cluster_kernel(const float4* __restrict__ x, const float4* __restrict__ dy, const float* __restrict__ gamma,
                      const float* __restrict__ beta, const float* __restrict__ stats, const float4* __restrict__ addend,
                      float4* __restrict__ dx, float* __restrict__ dgamma, float* __restrict__ dbeta, int64_t rows, int C,
                      int cgc, int64_t rows_per_cta, float floor, int early_x)
{
    namespace cgr = cooperative_groups;
    cgr::cluster_group cluster = cgr::this_cluster();
    __shared__ float wpart[kBnThreads / 32][kBnClusterMaxCgc * 8];
    __shared__ float part[kBnClusterMaxCgc * 8];
    __shared__ float coefs[kBnClusterMaxCgc * 8];
    pdl_launch_dependents();
    const int t = threadIdx.x;
    const unsigned int rank = cluster.block_rank();
    const int cl = blockIdx.x / kBnCluster;
    const int cg_total = C / 4;
    const int rl = kBnThreads / cgc;
    const int my_cg = t % cgc, my_rl = t / cgc;
    const int cg = cl * cgc + my_cg;
    const int64_t r0 = (int64_t)rank * rows_per_cta;
    int64_t r1 = r0 + rows_per_cta;
    if (r1 > rows) r1 = rows;
    int n = r1 > r0 + my_rl ? (int)((r1 - r0 - my_rl + rl - 1) / rl) : 0;
    if (n > NV) n = NV;                                     // the launcher sizes NV so that this never cuts
    const int64_t base = (r0 + my_rl) * cg_total + cg, step = (int64_t)rl * cg_total;

    if (!early_x) pdl_wait();
    const float4 mu = __ldg(reinterpret_cast<const float4*>(stats) + cg);
    const float4 rs = __ldg(reinterpret_cast<const float4*>(stats + C) + cg);
    const float4 gm = __ldg(reinterpret_cast<const float4*>(gamma) + cg);
    const float4 bt = __ldg(reinterpret_cast<const float4*>(beta) + cg);
    float4 xv[NV], dv[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) if (k < n) xv[k] = __ldg(x + base + k * step);
    if (early_x) pdl_wait();
#pragma unroll
    for (int k = 0; k < NV; ++k) if (k < n) dv[k] = __ldcg(dy + base + k * step);   // not the read-only path: such a load may be moved above the wait

    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        if (k < n) {
            float xh, dz;
            xh = bn_xhat(xv[k].x, mu.x, rs.x); dz = bn_z(xh, gm.x, bt.x) > floor ? dv[k].x : 0.f; a.x += dz; b.x = fmaf(dz, xh, b.x);
            xv[k].x = xh; dv[k].x = dz;
            xh = bn_xhat(xv[k].y, mu.y, rs.y); dz = bn_z(xh, gm.y, bt.y) > floor ? dv[k].y : 0.f; a.y += dz; b.y = fmaf(dz, xh, b.y);
            xv[k].y = xh; dv[k].y = dz;
            xh = bn_xhat(xv[k].z, mu.z, rs.z); dz = bn_z(xh, gm.z, bt.z) > floor ? dv[k].z : 0.f; a.z += dz; b.z = fmaf(dz, xh, b.z);
            xv[k].z = xh; dv[k].z = dz;
            xh = bn_xhat(xv[k].w, mu.w, rs.w); dz = bn_z(xh, gm.w, bt.w) > floor ? dv[k].w : 0.f; a.w += dz; b.w = fmaf(dz, xh, b.w);
            xv[k].w = xh; dv[k].w = dz;
        }
    }
    // row lanes of one column group inside a warp: fixed butterfly; then the warps in ascending order
    for (int off = 16; off >= cgc; off >>= 1) {
        a.x += __shfl_xor_sync(0xffffffffu, a.x, off); a.y += __shfl_xor_sync(0xffffffffu, a.y, off);
        a.z += __shfl_xor_sync(0xffffffffu, a.z, off); a.w += __shfl_xor_sync(0xffffffffu, a.w, off);
        b.x += __shfl_xor_sync(0xffffffffu, b.x, off); b.y += __shfl_xor_sync(0xffffffffu, b.y, off);
        b.z += __shfl_xor_sync(0xffffffffu, b.z, off); b.w += __shfl_xor_sync(0xffffffffu, b.w, off);
    }
    const int warp = t >> 5, lane = t & 31;
    if (lane < cgc) {
        float* d = &wpart[warp][lane * 8];
        d[0] = a.x; d[1] = a.y; d[2] = a.z; d[3] = a.w; d[4] = b.x; d[5] = b.y; d[6] = b.z; d[7] = b.w;
    }
    __syncthreads();
    if (t < cgc * 8) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kBnThreads / 32; ++w) s += wpart[w][t];
        part[t] = s;
    }
    cluster.sync();
    if (t < cgc * 8) {
        double s = 0.0;
#pragma unroll
        for (unsigned int r = 0; r < (unsigned int)kBnCluster; ++r) s += (double)*cluster.map_shared_rank(&part[t], r);
        coefs[t] = (float)(s * (1.0 / (double)rows));
        if (rank == 0) {
            const int c = (cl * cgc + (t >> 3)) * 4 + (t & 3);
            if (t & 4) dgamma[c] = (float)s; else dbeta[c] = (float)s;
        }
    }
    __syncthreads();
    cluster.barrier_arrive();                               // this CTA no longer reads the others' shared memory
    const float4 ca = *reinterpret_cast<const float4*>(&coefs[my_cg * 8]);
    const float4 cb = *reinterpret_cast<const float4*>(&coefs[my_cg * 8 + 4]);
    const float4 sc = make_float4(gm.x * rs.x, gm.y * rs.y, gm.z * rs.z, gm.w * rs.w);
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        if (k < n) {
            const int64_t i = base + k * step;
            float4 o;
            o.x = sc.x * (dv[k].x - ca.x - xv[k].x * cb.x);
            o.y = sc.y * (dv[k].y - ca.y - xv[k].y * cb.y);
            o.z = sc.z * (dv[k].z - ca.z - xv[k].z * cb.z);
            o.w = sc.w * (dv[k].w - ca.w - xv[k].w * cb.w);
            if (ADDEND) { const float4 e = __ldcg(addend + i); o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            if (ACCUM) { const float4 e = dx[i]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            dx[i] = o;
        }
    }
    cluster.barrier_wait();                                 // shared memory stays alive until every CTA has read it
}

// The forward twin: statistics and y = max(gamma * xhat + beta, floor) in one launch, x read once into registers.
// Sums are shifted by the tensor's first row (the same shift in every CTA, so the partial sums add up).
template <int NV>
__global__ void __launch_bounds__(kBnThreads)
bn_fwd_cluster_kernel(const float4* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta, float eps,
                      float4* __restrict__ y, float* __restrict__ stats, int64_t rows, int C, int cgc, int64_t rows_per_cta,
                      float floor)
{
    namespace cgr = cooperative_groups;
    cgr::cluster_group cluster = cgr::this_cluster();
    __shared__ float wpart[kBnThreads / 32][kBnClusterMaxCgc * 8];
    __shared__ float part[kBnClusterMaxCgc * 8];
    __shared__ float coefs[kBnClusterMaxCgc * 8];
    pdl_launch_dependents();
    pdl_wait();
    const int t = threadIdx.x;
    const unsigned int rank = cluster.block_rank();
    const int cl = blockIdx.x / kBnCluster;
    const int cg_total = C / 4;
    const int rl = kBnThreads / cgc;
    const int my_cg = t % cgc, my_rl = t / cgc;
    const int cg = cl * cgc + my_cg;
    const int64_t r0 = (int64_t)rank * rows_per_cta;
    int64_t r1 = r0 + rows_per_cta;
    if (r1 > rows) r1 = rows;
    int n = r1 > r0 + my_rl ? (int)((r1 - r0 - my_rl + rl - 1) / rl) : 0;
    if (n > NV) n = NV;
    const int64_t base = (r0 + my_rl) * cg_total + cg, step = (int64_t)rl * cg_total;
    const float4 p0 = __ldcg(x + cg);                                              // shift = first row
    const float4 gm = __ldg(reinterpret_cast<const float4*>(gamma) + cg);
    const float4 bt = __ldg(reinterpret_cast<const float4*>(beta) + cg);
    float4 xv[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) if (k < n) xv[k] = __ldcg(x + base + k * step);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        if (k < n) {
            float d;
            d = xv[k].x - p0.x; a.x += d; b.x = fmaf(d, d, b.x);
            d = xv[k].y - p0.y; a.y += d; b.y = fmaf(d, d, b.y);
            d = xv[k].z - p0.z; a.z += d; b.z = fmaf(d, d, b.z);
            d = xv[k].w - p0.w; a.w += d; b.w = fmaf(d, d, b.w);
        }
    }
    for (int off = 16; off >= cgc; off >>= 1) {
        a.x += __shfl_xor_sync(0xffffffffu, a.x, off); a.y += __shfl_xor_sync(0xffffffffu, a.y, off);
        a.z += __shfl_xor_sync(0xffffffffu, a.z, off); a.w += __shfl_xor_sync(0xffffffffu, a.w, off);
        b.x += __shfl_xor_sync(0xffffffffu, b.x, off); b.y += __shfl_xor_sync(0xffffffffu, b.y, off);
        b.z += __shfl_xor_sync(0xffffffffu, b.z, off); b.w += __shfl_xor_sync(0xffffffffu, b.w, off);
    }
    const int warp = t >> 5, lane = t & 31;
    if (lane < cgc) {
        float* d = &wpart[warp][lane * 8];
        d[0] = a.x; d[1] = a.y; d[2] = a.z; d[3] = a.w; d[4] = b.x; d[5] = b.y; d[6] = b.z; d[7] = b.w;
    }
    __syncthreads();
    if (t < cgc * 8) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kBnThreads / 32; ++w) s += wpart[w][t];
        part[t] = s;
    }
    cluster.sync();
    if (t < cgc * 4) {                                      // one thread per channel of the slice: (group, element)
        const int cgl = t >> 2, e = t & 3;
        double sa = 0.0, sb = 0.0;
#pragma unroll
        for (unsigned int r = 0; r < (unsigned int)kBnCluster; ++r) {
            const float* rp = cluster.map_shared_rank(&part[cgl * 8], r);
            sa += (double)rp[e]; sb += (double)rp[4 + e];
        }
        const int c = (cl * cgc + cgl) * 4 + e;
        const double inv_rows = 1.0 / (double)rows;
        const double shift = (double)__ldcg(reinterpret_cast<const float*>(x) + c);
        const double ms = sa * inv_rows;
        double var = sb * inv_rows - ms * ms;
        if (var < 0.0) var = 0.0;
        const float mean = (float)(shift + ms), rstd = (float)(1.0 / sqrt(var + (double)eps));
        coefs[cgl * 8 + e] = mean; coefs[cgl * 8 + 4 + e] = rstd;
        if (rank == 0) { stats[c] = mean; stats[C + c] = rstd; }
    }
    __syncthreads();
    cluster.barrier_arrive();
    const float4 mu = *reinterpret_cast<const float4*>(&coefs[my_cg * 8]);
    const float4 rs = *reinterpret_cast<const float4*>(&coefs[my_cg * 8 + 4]);
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        if (k < n) {
            float4 o;
            o.x = fmaxf(bn_z(bn_xhat(xv[k].x, mu.x, rs.x), gm.x, bt.x), floor);
            o.y = fmaxf(bn_z(bn_xhat(xv[k].y, mu.y, rs.y), gm.y, bt.y), floor);
            o.z = fmaxf(bn_z(bn_xhat(xv[k].z, mu.z, rs.z), gm.z, bt.z), floor);
            o.w = fmaxf(bn_z(bn_xhat(xv[k].w, mu.w, rs.w), gm.w, bt.w), floor);
            y[base + k * step] = o;
        }
    }
    cluster.barrier_wait();
}

struct BnClusterPlan { bool ok; int cgc, n_clusters, nv; int64_t rows_per_cta; };

// Eligible: micro-batch sized tensors whose rows fit the registers of kBnCluster CTAs per column-group slice.  Prefers few
// rows per thread (more CTAs pulling on memory), then wide slices (longer contiguous segments per row).
BnClusterPlan bn_cluster_plan(int64_t rows, int C)
{
    BnClusterPlan p = {false, 0, 0, 0, 0};
    if (C % 4 != 0 || rows < 1 || rows * C > (int64_t)(2 << 20)) return p;
    const int cg_total = C / 4;
    const int64_t rpc = ceil_div64(rows, kBnCluster);
    static const int prefs[3] = {2, 4, 8};
    for (int pi = 0; pi < 3; ++pi) {
        for (int cgc = kBnClusterMaxCgc; cgc >= 2; cgc >>= 1) {       // a slice of one 16-byte group per row was tried: slower (half-used sectors)
            if (cg_total % cgc != 0) continue;
            const int n_clusters = cg_total / cgc;
            if (n_clusters > kBnClusterMaxActive) continue;
            const int64_t nv = ceil_div64(rpc, kBnThreads / cgc);
            if (nv > prefs[pi]) continue;
            p.ok = true; p.cgc = cgc; p.n_clusters = n_clusters; p.rows_per_cta = rpc;
            p.nv = nv <= 1 ? 1 : nv <= 2 ? 2 : nv <= 4 ? 4 : 8;
            return p;
        }
    }
    return p;
}

// ------------------------------------------------------------------------------------------------
// BN on tensors of 8 MB and more (batch-sized tensors, 56x56 maps): bandwidth, not latency, is the limit.
//   reduce: one resident wave of CTAs streams the rows (eight 128-bit loads in flight per thread); the CTAs of a cluster
//           add their per-channel sums through distributed shared memory, so that only a few dozen partial rows reach
//           global memory and no CTA stays behind to combine hundreds of them;
//   apply:  every CTA adds those few partials itself (fp64, fixed order) in its prologue - no ticket, no fence, no
//           statistics round trip between the two kernels - then streams its rows; CTA 0 stores the statistics /
//           parameter gradients.  The apply kernel walks its slab from the end: the rows the reduce kernel read last
//           are the ones still in L2.
// ------------------------------------------------------------------------------------------------
constexpr int kBnBigCluster = 8;
#ifndef HPF_BN_NB_F
#define HPF_BN_NB_F 4           // rows per batch of loads: forward kernels (one operand)
#endif
#ifndef HPF_BN_NB_B
#define HPF_BN_NB_B 2           // backward kernels (two operands)
#endif
constexpr int kBnBigMaxPartials = 37;            // 296 CTAs in clusters of 8

template <bool BWD>
__global__ void __launch_bounds__(kBnThreads, 2)
bn_reduce_big_kernel(const float4* __restrict__ x4, const float4* __restrict__ dy4, const float* __restrict__ gamma,
                     const float* __restrict__ beta, const float* __restrict__ stats, int64_t rows, int C, int cgt, int rl,
                     int64_t rows_per_blk, float* __restrict__ partials, float floor)
{
    namespace cgr = cooperative_groups;
    cgr::cluster_group cluster = cgr::this_cluster();
    __shared__ float sh[kBnThreads][8];
    __shared__ float part[kBnThreads * 8];
    pdl_launch_dependents();
    pdl_wait();
    const int t = threadIdx.x;
    const int cg_total = C / 4;                  // == cgt: one pass
    const int my_rl = t / cgt, my_cg = t % cgt;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_blk;
    int64_t r1 = r0 + rows_per_blk;
    if (r1 > rows) r1 = rows;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    {
        float4 p0, p1, gm, bt;
        if (BWD) {
            p0 = __ldg(reinterpret_cast<const float4*>(stats) + my_cg);
            p1 = __ldg(reinterpret_cast<const float4*>(stats + C) + my_cg);
            gm = __ldg(reinterpret_cast<const float4*>(gamma) + my_cg);
            bt = __ldg(reinterpret_cast<const float4*>(beta) + my_cg);
        } else {
            p0 = __ldg(x4 + my_cg);                                                   // shift = first row
        }
        const float4* xp = x4 + (r0 + my_rl) * cg_total + my_cg;
        const float4* dp = dy4 + (r0 + my_rl) * cg_total + my_cg;
        const int64_t step = (int64_t)rl * cg_total;
        const int n = r1 > r0 + my_rl ? (int)((r1 - r0 - my_rl + rl - 1) / rl) : 0;
        // batches of predicated loads: every load of a batch is in flight before the first use (a scalar remainder
        // loop would pay one memory round trip per row)
        constexpr int NB = BWD ? HPF_BN_NB_B : HPF_BN_NB_F;
        for (int k0 = 0; k0 < n; k0 += NB) {
            float4 v[NB], g[BWD ? NB : 1];
#pragma unroll
            for (int j = 0; j < NB; ++j) if (k0 + j < n) v[j] = __ldg(xp + (k0 + j) * step);
            if (BWD) {
#pragma unroll
                for (int j = 0; j < NB; ++j) if (k0 + j < n) g[j] = __ldg(dp + (k0 + j) * step);
            }
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                if (k0 + j < n) {
                    if (BWD) {
                        float xh, dz;
                        xh = bn_xhat(v[j].x, p0.x, p1.x); dz = bn_z(xh, gm.x, bt.x) > floor ? g[j].x : 0.f; a.x += dz; b.x = fmaf(dz, xh, b.x);
                        xh = bn_xhat(v[j].y, p0.y, p1.y); dz = bn_z(xh, gm.y, bt.y) > floor ? g[j].y : 0.f; a.y += dz; b.y = fmaf(dz, xh, b.y);
                        xh = bn_xhat(v[j].z, p0.z, p1.z); dz = bn_z(xh, gm.z, bt.z) > floor ? g[j].z : 0.f; a.z += dz; b.z = fmaf(dz, xh, b.z);
                        xh = bn_xhat(v[j].w, p0.w, p1.w); dz = bn_z(xh, gm.w, bt.w) > floor ? g[j].w : 0.f; a.w += dz; b.w = fmaf(dz, xh, b.w);
                    } else {
                        float d;
                        d = v[j].x - p0.x; a.x += d; b.x = fmaf(d, d, b.x);
                        d = v[j].y - p0.y; a.y += d; b.y = fmaf(d, d, b.y);
                        d = v[j].z - p0.z; a.z += d; b.z = fmaf(d, d, b.z);
                        d = v[j].w - p0.w; a.w += d; b.w = fmaf(d, d, b.w);
                    }
                }
            }
        }
    }
    // the CTA's sums per channel: row lanes in a fixed order
    if (cgt <= 16) {
        for (int off = 16; off >= cgt; off >>= 1) {
            a.x += __shfl_xor_sync(0xffffffffu, a.x, off); a.y += __shfl_xor_sync(0xffffffffu, a.y, off);
            a.z += __shfl_xor_sync(0xffffffffu, a.z, off); a.w += __shfl_xor_sync(0xffffffffu, a.w, off);
            b.x += __shfl_xor_sync(0xffffffffu, b.x, off); b.y += __shfl_xor_sync(0xffffffffu, b.y, off);
            b.z += __shfl_xor_sync(0xffffffffu, b.z, off); b.w += __shfl_xor_sync(0xffffffffu, b.w, off);
        }
        const int warp = t >> 5, lane = t & 31;
        if (lane < cgt) {
            float* d = sh[warp * cgt + lane];
            d[0] = a.x; d[1] = a.y; d[2] = a.z; d[3] = a.w; d[4] = b.x; d[5] = b.y; d[6] = b.z; d[7] = b.w;
        }
        __syncthreads();
        if (t < cgt * 8) {
            const int cgl = t >> 3, comp = t & 7;
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kBnThreads / 32; ++w) s += sh[w * cgt + cgl][comp];
            part[t] = s;
        }
    } else {
        sh[t][0] = a.x; sh[t][1] = a.y; sh[t][2] = a.z; sh[t][3] = a.w;
        sh[t][4] = b.x; sh[t][5] = b.y; sh[t][6] = b.z; sh[t][7] = b.w;
        __syncthreads();
        for (int o = t; o < cgt * 8; o += kBnThreads) {
            const int cgl = o >> 3, comp = o & 7;
            float s = 0.f;
            for (int l = 0; l < rl; ++l) s += sh[l * cgt + cgl][comp];
            part[o] = s;
        }
    }
    cluster.sync();
    // rank r adds the cluster's CTAs (ascending) for its eighth of the (channel group, component) pairs
    const unsigned int rank = cluster.block_rank();
    const int cl = blockIdx.x / kBnBigCluster;
    for (int o = (int)rank * cgt + t; o < ((int)rank + 1) * cgt; o += kBnThreads) {
        float s = 0.f;
#pragma unroll
        for (unsigned int r = 0; r < (unsigned int)kBnBigCluster; ++r) s += *cluster.map_shared_rank(&part[o], r);
        const int cgl = o >> 3, comp = o & 7;
        partials[((int64_t)cl * 2 + (comp >> 2)) * C + cgl * 4 + (comp & 3)] = s;
    }
    cluster.sync();
}

// Prologue of the big apply kernels: per-channel totals of the n_part partial rows (fp64, ascending), then the forward
// statistics (mean, rstd) or the backward coefficients (sum dz / rows, sum dz*xhat / rows) into fin[0][c], fin[1][c].
template <bool BWD>
__device__ __forceinline__ void bn_big_finalise(const float* __restrict__ partials, int n_part, int64_t rows, int C, int cgt, int rl,
                                                float eps, const float* __restrict__ x, float* __restrict__ out_a,
                                                float* __restrict__ out_b, bool write_out, double (*shd)[8], float* fin)
{
    const int t = threadIdx.x;
    const int my_rl = t / cgt, my_cg = t % cgt;
    double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
    // four partial rows per batch, their eight loads in flight together
    for (int k0 = my_rl; k0 < n_part; k0 += 4 * rl) {
        float4 va[4], vb[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = k0 + j * rl;
            const bool in = k < n_part;
            va[j] = in ? __ldcg(reinterpret_cast<const float4*>(partials + ((int64_t)k * 2 + 0) * C) + my_cg) : make_float4(0.f, 0.f, 0.f, 0.f);
            vb[j] = in ? __ldcg(reinterpret_cast<const float4*>(partials + ((int64_t)k * 2 + 1) * C) + my_cg) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            acc[0] += (double)va[j].x; acc[1] += (double)va[j].y; acc[2] += (double)va[j].z; acc[3] += (double)va[j].w;
            acc[4] += (double)vb[j].x; acc[5] += (double)vb[j].y; acc[6] += (double)vb[j].z; acc[7] += (double)vb[j].w;
        }
    }
    if (cgt <= 16) {
        for (int off = 16; off >= cgt; off >>= 1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], off);
        }
        const int warp = t >> 5, lane = t & 31;
        double (*wsum)[8] = shd + kBnThreads / 2;
        if (lane < cgt) {
#pragma unroll
            for (int j = 0; j < 8; ++j) wsum[warp * cgt + lane][j] = acc[j];
        }
        __syncthreads();
        if (t < cgt * 8) {
            const int cgl = t >> 3, comp = t & 7;
            double s = 0.0;
            for (int w = 0; w < kBnThreads / 32; ++w) s += wsum[w * cgt + cgl][comp];
            shd[cgl][comp] = s;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) shd[t][j] = acc[j];
        __syncthreads();
        double s[8];
        const bool mine = t < cgt;                 // thread t < cgt totals column group t (all eight components)
        if (mine) {
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = 0.0;
            for (int l = 0; l < rl; ++l) {
#pragma unroll
                for (int j = 0; j < 8; ++j) s[j] += shd[l * cgt + t][j];
            }
        }
        __syncthreads();
        if (mine) {
#pragma unroll
            for (int j = 0; j < 8; ++j) shd[t][j] = s[j];
        }
    }
    __syncthreads();
    const double inv_rows = 1.0 / (double)rows;
    for (int cl = t; cl < cgt * 4; cl += kBnThreads) {
        const int cgl = cl >> 2, e = cl & 3;
        const double sa = shd[cgl][e], sb = shd[cgl][4 + e];
        if (BWD) {
            fin[cl] = (float)(sa * inv_rows);
            fin[C + cl] = (float)(sb * inv_rows);
            if (write_out) { out_a[cl] = (float)sa; out_b[cl] = (float)sb; }        // dbeta, dgamma
        } else {
            const double shift = (double)__ldg(x + cl);
            const double ms = sa * inv_rows;
            double var = sb * inv_rows - ms * ms;
            if (var < 0.0) var = 0.0;
            const float mean = (float)(shift + ms), rstd = (float)(1.0 / sqrt(var + (double)eps));
            fin[cl] = mean; fin[C + cl] = rstd;
            if (write_out) { out_a[cl] = mean; out_b[cl] = rstd; }
        }
    }
    __syncthreads();
}

// dynamic shared memory of the big apply kernels: [512][8] doubles for the prologue, then 2*C floats
inline size_t bn_big_apply_smem(int C) { return (size_t)kBnThreads * 8 * sizeof(double) + 2 * (size_t)C * sizeof(float); }

__global__ void __launch_bounds__(kBnThreads, 2)
bn_apply_big_fwd_kernel(const float4* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                        const float* __restrict__ partials, int n_part, float eps, float* __restrict__ stats,
                        float4* __restrict__ y, int64_t rows, int C, int cgt, int rl, int64_t rows_per_blk, float floor, int stream_out)
{
    extern __shared__ __align__(16) unsigned char bn_big_smem[];
    double (*shd)[8] = reinterpret_cast<double (*)[8]>(bn_big_smem);
    float* fin = reinterpret_cast<float*>(bn_big_smem + (size_t)kBnThreads * 8 * sizeof(double));
    pdl_launch_dependents();
    pdl_wait();
    bn_big_finalise<false>(partials, n_part, rows, C, cgt, rl, eps, reinterpret_cast<const float*>(x), stats, stats + C,
                           blockIdx.x == 0, shd, fin);
    const int t = threadIdx.x, cg_total = C / 4;
    const int my_rl = t / cgt, my_cg = t % cgt;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_blk;
    int64_t r1 = r0 + rows_per_blk;
    if (r1 > rows) r1 = rows;
    const float4 mu = *reinterpret_cast<const float4*>(fin + my_cg * 4);
    const float4 rs = *reinterpret_cast<const float4*>(fin + C + my_cg * 4);
    const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + my_cg);
    const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + my_cg);
    const int64_t base = (r0 + my_rl) * cg_total + my_cg, step = (int64_t)rl * cg_total;
    const int n = r1 > r0 + my_rl ? (int)((r1 - r0 - my_rl + rl - 1) / rl) : 0;
    constexpr int NB = HPF_BN_NB_F;
    for (int k0 = n - 1; k0 >= 0; k0 -= NB) {              // from the end of the slab, in batches of predicated loads
        float4 v[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) if (k0 - j >= 0) v[j] = __ldg(x + base + (k0 - j) * step);
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            if (k0 - j >= 0) {
                float4 o;
                o.x = fmaxf(bn_z(bn_xhat(v[j].x, mu.x, rs.x), g.x, b.x), floor);
                o.y = fmaxf(bn_z(bn_xhat(v[j].y, mu.y, rs.y), g.y, b.y), floor);
                o.z = fmaxf(bn_z(bn_xhat(v[j].z, mu.z, rs.z), g.z, b.z), floor);
                o.w = fmaxf(bn_z(bn_xhat(v[j].w, mu.w, rs.w), g.w, b.w), floor);
                if (stream_out) __stcs(y + base + (k0 - j) * step, o); else y[base + (k0 - j) * step] = o;
            }
        }
    }
}

template <bool ADDEND, bool ACCUM>
__global__ void __launch_bounds__(kBnThreads, 2)
bn_apply_big_bwd_kernel(const float4* __restrict__ x, const float4* __restrict__ dy, const float* __restrict__ gamma,
                        const float* __restrict__ beta, const float* __restrict__ stats, const float* __restrict__ partials,
                        int n_part, float* __restrict__ dgamma, float* __restrict__ dbeta, const float4* __restrict__ addend,
                        float4* __restrict__ dx, int64_t rows, int C, int cgt, int rl, int64_t rows_per_blk, float floor, int stream_out)
{
    extern __shared__ __align__(16) unsigned char bn_big_smem[];
    double (*shd)[8] = reinterpret_cast<double (*)[8]>(bn_big_smem);
    float* fin = reinterpret_cast<float*>(bn_big_smem + (size_t)kBnThreads * 8 * sizeof(double));
    pdl_launch_dependents();
    pdl_wait();
    bn_big_finalise<true>(partials, n_part, rows, C, cgt, rl, 0.f, nullptr, dbeta, dgamma, blockIdx.x == 0, shd, fin);
    const int t = threadIdx.x, cg_total = C / 4;
    const int my_rl = t / cgt, my_cg = t % cgt;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_blk;
    int64_t r1 = r0 + rows_per_blk;
    if (r1 > rows) r1 = rows;
    const float4 ca = *reinterpret_cast<const float4*>(fin + my_cg * 4);
    const float4 cb = *reinterpret_cast<const float4*>(fin + C + my_cg * 4);
    const float4 mu = __ldg(reinterpret_cast<const float4*>(stats) + my_cg);
    const float4 rs = __ldg(reinterpret_cast<const float4*>(stats + C) + my_cg);
    const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + my_cg);
    const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + my_cg);
    const int64_t base = (r0 + my_rl) * cg_total + my_cg, step = (int64_t)rl * cg_total;
    const int n = r1 > r0 + my_rl ? (int)((r1 - r0 - my_rl + rl - 1) / rl) : 0;
    constexpr int NB = HPF_BN_NB_B;
    for (int k0 = n - 1; k0 >= 0; k0 -= NB) {
        float4 v[NB], d[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) if (k0 - j >= 0) { v[j] = __ldg(x + base + (k0 - j) * step); d[j] = __ldg(dy + base + (k0 - j) * step); }
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            if (k0 - j >= 0) {
                const int64_t i = base + (k0 - j) * step;
                float4 o;
                o.x = bn_dx1(v[j].x, d[j].x, mu.x, rs.x, g.x, b.x, ca.x, cb.x, floor);
                o.y = bn_dx1(v[j].y, d[j].y, mu.y, rs.y, g.y, b.y, ca.y, cb.y, floor);
                o.z = bn_dx1(v[j].z, d[j].z, mu.z, rs.z, g.z, b.z, ca.z, cb.z, floor);
                o.w = bn_dx1(v[j].w, d[j].w, mu.w, rs.w, g.w, b.w, ca.w, cb.w, floor);
                if (ADDEND) { const float4 e = __ldg(addend + i); o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
                if (ACCUM) { const float4 e = dx[i]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
                if (stream_out) __stcs(dx + i, o); else dx[i] = o;
            }
        }
    }
}

struct BnBigPlan { bool ok; int n_clusters, nblk_apply, stream_out; int64_t rows_per_blk, rows_per_blk_apply; };

// Clusters of the reduce kernel that are resident together on this device (asked once per kernel).
template <bool BWD>
int bn_big_max_clusters()
{
    // per device: a process may drive several GPUs, and the answer (like the attributes set below) belongs to one of them
    static int cached_by_device[64];
    static bool have[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 0; }
    if (have[dev]) return cached_by_device[dev];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kBnBigCluster * kBnBigMaxPartials); cfg.blockDim = dim3(kBnThreads);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kBnBigCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, bn_reduce_big_kernel<BWD>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    cached_by_device[dev] = n; have[dev] = true;
    return n;
}

template <bool BWD>
BnBigPlan bn_big_plan(int64_t rows, int C, const BnPlan& p)
{
    BnBigPlan b = {false, 0, 0, 0, 0, 0};
    if (!g_bn_cluster || C % 4 != 0 || p.passes != 1 || (p.cgt & (p.cgt - 1)) != 0) return b;   // power of two: cgt * rl == block
    // large tensors, and wide ones (2048 channels: one row lane per block, so the last block of the ticket scheme would
    // add its hundred partial rows one after the other)
    if (rows * C < kBnLargeElems && p.nblk <= 16 * p.rl) return b;
    int ncl = bn_big_max_clusters<BWD>();
    if (ncl > kBnBigMaxPartials) ncl = kBnBigMaxPartials;
    const int64_t want = rows / ((int64_t)p.rl * 8 * kBnBigCluster);          // at least eight rows per thread
    if (want < ncl) ncl = (int)want;
    if (ncl < 2 || ncl > p.nblk) return b;                                    // the scratch holds p.nblk partial rows
    b.ok = true; b.n_clusters = ncl;
    b.rows_per_blk = ceil_div64(rows, (int64_t)ncl * kBnBigCluster);
    int64_t na = rows / ((int64_t)p.rl * 8);
    if (na > 2 * 148) na = 2 * 148;
    if (na < 1) na = 1;
    b.rows_per_blk_apply = ceil_div64(rows, na);
    b.nblk_apply = (int)ceil_div64(rows, b.rows_per_blk_apply);
    b.stream_out = rows * C * (int64_t)sizeof(float) > (int64_t)(48 << 20) ? 1 : 0;   // input + output beyond L2: do not keep the output   // input + output beyond L2: do not keep the output
    return b;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_cluster_pdl(void (*kernel)(KArgs...), int grid, int block, int cluster, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = g_pdl_enabled ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int ew_blocks(int64_t n_items)
{
    int64_t nb = ceil_div64(n_items, kThreads);
    if (nb > kMaxBlocks * 4) nb = kMaxBlocks * 4;
    if (nb < 1) nb = 1;
    return (int)nb;
}

// ------------------------------------------------------------------------------------------------
// element-wise
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
add_kernel(const float* __restrict__ a, const float* __restrict__ b, float* __restrict__ out, int64_t n)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t n4 = n / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = t0; i < n4; i += stride) {
        const float4 u = __ldg(reinterpret_cast<const float4*>(a) + i), v = __ldg(reinterpret_cast<const float4*>(b) + i);
        reinterpret_cast<float4*>(out)[i] = make_float4(u.x + v.x, u.y + v.y, u.z + v.z, u.w + v.w);
    }
    for (int64_t i = n4 * 4 + t0; i < n; i += stride) out[i] = a[i] + b[i];
}

// Stand-alone ReLU (the post-activation residual block ends in one): y = max(x, 0); dx = dy * [x > 0] (+ addend) (+= dx).
__global__ void __launch_bounds__(kThreads)
relu_fwd_kernel(const float* __restrict__ x, float* __restrict__ y, int64_t n)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t n4 = n / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = t0; i < n4; i += stride) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(x) + i);
        reinterpret_cast<float4*>(y)[i] = make_float4(fmaxf(v.x, 0.f), fmaxf(v.y, 0.f), fmaxf(v.z, 0.f), fmaxf(v.w, 0.f));
    }
    for (int64_t i = n4 * 4 + t0; i < n; i += stride) y[i] = fmaxf(x[i], 0.f);
}

template <bool ADDEND, bool ACCUM>
__global__ void __launch_bounds__(kThreads)
relu_bwd_kernel(const float* __restrict__ x, const float* __restrict__ dy, const float* __restrict__ addend,
                float* __restrict__ dx, int64_t n)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t n4 = n / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = t0; i < n4; i += stride) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(x) + i), d = __ldg(reinterpret_cast<const float4*>(dy) + i);
        float4 o = make_float4(v.x > 0.f ? d.x : 0.f, v.y > 0.f ? d.y : 0.f, v.z > 0.f ? d.z : 0.f, v.w > 0.f ? d.w : 0.f);
        if (ADDEND) { const float4 e = __ldg(reinterpret_cast<const float4*>(addend) + i); o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
        if (ACCUM) { const float4 e = reinterpret_cast<const float4*>(dx)[i]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
        reinterpret_cast<float4*>(dx)[i] = o;
    }
    for (int64_t i = n4 * 4 + t0; i < n; i += stride) {
        float o = x[i] > 0.f ? dy[i] : 0.f;
        if (ADDEND) o += addend[i];
        if (ACCUM) o += dx[i];
        dx[i] = o;
    }
}

template <bool ACCUM>
__global__ void __launch_bounds__(kThreads)
accumulate_kernel(float* __restrict__ dst, const float* __restrict__ src, int64_t n)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t n4 = n / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = t0; i < n4; i += stride) {
        float4 v = __ldg(reinterpret_cast<const float4*>(src) + i);
        if (ACCUM) { const float4 e = reinterpret_cast<float4*>(dst)[i]; v.x += e.x; v.y += e.y; v.z += e.z; v.w += e.w; }
        reinterpret_cast<float4*>(dst)[i] = v;
    }
    for (int64_t i = n4 * 4 + t0; i < n; i += stride) dst[i] = ACCUM ? dst[i] + src[i] : src[i];
}

// out[j] = (slots[0][j] + slots[1][j] + ... + slots[M-1][j]) / M, ascending m.  Reads M*G floats,
// writes G: pure streaming.  Slot m starts at m*G floats, so the widest aligned access depends on G:
// VEC = 4 when G % 4 == 0, 2 when G is even, else 1.
template <int VEC>
__global__ void __launch_bounds__(kThreads)
grad_average_kernel(const float* __restrict__ slots, float* __restrict__ out, int M, int64_t G, float inv_m)
{
    const int64_t nv = G / VEC;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += stride) {
        float s[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) s[e] = 0.f;
        // eight slots per batch, the loads of a batch in flight together whatever M is (a partially unrolled loop would
        // run its remainder one load at a time); the sum stays in ascending slot order
        for (int m0 = 0; m0 < M; m0 += 8) {
            float q[8][VEC];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (m0 + j < M) {
                    const float* src = slots + (int64_t)(m0 + j) * G + i * VEC;
                    if (VEC == 4) { const float4 v = __ldcs(reinterpret_cast<const float4*>(src)); q[j][0] = v.x; q[j][1 % VEC] = v.y; q[j][2 % VEC] = v.z; q[j][3 % VEC] = v.w; }
                    else if (VEC == 2) { const float2 v = __ldcs(reinterpret_cast<const float2*>(src)); q[j][0] = v.x; q[j][1 % VEC] = v.y; }
                    else q[j][0] = __ldcs(src);
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (m0 + j < M) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) s[e] += q[j][e];
                }
            }
        }
        float* dst = out + i * VEC;
        if (VEC == 4) *reinterpret_cast<float4*>(dst) = make_float4(s[0] * inv_m, s[1 % VEC] * inv_m, s[2 % VEC] * inv_m, s[3 % VEC] * inv_m);
        else if (VEC == 2) *reinterpret_cast<float2*>(dst) = make_float2(s[0] * inv_m, s[1 % VEC] * inv_m);
        else dst[0] = s[0] * inv_m;
    }
}

// Gradient average fused with the parameter update (Section 5.3: averaged gradients, then apply_gradients):
//   gbar = (sum_m g_m) / M (ascending m);  g' = gbar + wd * theta;  v <- mu * v - lr * g';  theta <- theta + v.
// One pass over the flat buffers: reads M slots + theta + v, writes gbar (optional) + theta + v.
template <int VEC>
__global__ void __launch_bounds__(kThreads)
sgd_momentum_kernel(const float* __restrict__ slots, float* __restrict__ gavg, float* __restrict__ theta,
                    float* __restrict__ vel, int M, int64_t G, float inv_m, float lr, float mu, float wd)
{
    const int64_t nv = G / VEC;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += stride) {
        float s[VEC], th[VEC], v[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) s[e] = 0.f;
        for (int m0 = 0; m0 < M; m0 += 8) {          // batches of eight slots, as in grad_average_kernel
            float q[8][VEC];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (m0 + j < M) {
                    const float* src = slots + (int64_t)(m0 + j) * G + i * VEC;
                    if (VEC == 4) { const float4 w4 = __ldcs(reinterpret_cast<const float4*>(src)); q[j][0] = w4.x; q[j][1 % VEC] = w4.y; q[j][2 % VEC] = w4.z; q[j][3 % VEC] = w4.w; }
                    else q[j][0] = __ldcs(src);
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (m0 + j < M) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) s[e] += q[j][e];
                }
            }
        }
        if (VEC == 4) {
            const float4 a = *reinterpret_cast<const float4*>(theta + i * 4), b = *reinterpret_cast<const float4*>(vel + i * 4);
            th[0] = a.x; th[1 % VEC] = a.y; th[2 % VEC] = a.z; th[3 % VEC] = a.w; v[0] = b.x; v[1 % VEC] = b.y; v[2 % VEC] = b.z; v[3 % VEC] = b.w;
        } else { th[0] = theta[i]; v[0] = vel[i]; }
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            s[e] *= inv_m;
            const float g = fmaf(wd, th[e], s[e]);
            v[e] = fmaf(mu, v[e], -lr * g);
            th[e] += v[e];
        }
        if (VEC == 4) {
            if (gavg) *reinterpret_cast<float4*>(gavg + i * 4) = make_float4(s[0], s[1 % VEC], s[2 % VEC], s[3 % VEC]);
            *reinterpret_cast<float4*>(theta + i * 4) = make_float4(th[0], th[1 % VEC], th[2 % VEC], th[3 % VEC]);
            *reinterpret_cast<float4*>(vel + i * 4) = make_float4(v[0], v[1 % VEC], v[2 % VEC], v[3 % VEC]);
        } else {
            if (gavg) gavg[i] = s[0];
            theta[i] = th[0]; vel[i] = v[0];
        }
    }
}

__global__ void stamp_kernel(unsigned long long* slot)
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    *slot = t;
}

__global__ void loss_average_kernel(const float* __restrict__ loss_slots, float* __restrict__ out, int M)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        float s = 0.f;
        for (int m = 0; m < M; ++m) s += loss_slots[m];
        *out = s / (float)M;
    }
}

// ------------------------------------------------------------------------------------------------
// max-pool (only the 224x224 layout uses it)
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
maxpool_fwd_kernel(const float* __restrict__ x, float* __restrict__ y, ConvShape s)
{
    const int64_t total = (int64_t)s.N * s.P * s.Q * s.C;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c = (int)(i % s.C);
        int64_t r = i / s.C;
        const int q = (int)(r % s.Q); r /= s.Q;
        const int p = (int)(r % s.P);
        const int n = (int)(r / s.P);
        float best = -INFINITY;
        for (int rr = 0; rr < s.R; ++rr) {
            const int ih = p * s.stride + rr - s.pad;
            if (ih < 0 || ih >= s.H) continue;
            for (int ss = 0; ss < s.R; ++ss) {
                const int iw = q * s.stride + ss - s.pad;
                if (iw < 0 || iw >= s.W) continue;
                best = fmaxf(best, __ldg(&x[(((int64_t)n * s.H + ih) * s.W + iw) * s.C + c]));
            }
        }
        y[i] = best;
    }
}

// Gather form (no atomics, fixed order): an input position receives dy of every window whose first
// maximum (row-major window order) it is.
template <bool ACCUM>
__global__ void __launch_bounds__(kThreads)
maxpool_bwd_kernel(const float* __restrict__ x, const float* __restrict__ dy, float* __restrict__ dx, ConvShape s)
{
    const int64_t total = (int64_t)s.N * s.H * s.W * s.C;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c = (int)(i % s.C);
        int64_t r = i / s.C;
        const int w = (int)(r % s.W); r /= s.W;
        const int h = (int)(r % s.H);
        const int n = (int)(r / s.H);
        const float mine = __ldg(&x[i]);
        float acc = 0.f;
        // windows (p,q) that contain (h,w): p*stride - pad <= h < p*stride - pad + R
        int p_lo = h + s.pad - s.R + 1; p_lo = p_lo <= 0 ? 0 : (p_lo + s.stride - 1) / s.stride;
        int p_hi = (h + s.pad) / s.stride; if (p_hi > s.P - 1) p_hi = s.P - 1;
        int q_lo = w + s.pad - s.R + 1; q_lo = q_lo <= 0 ? 0 : (q_lo + s.stride - 1) / s.stride;
        int q_hi = (w + s.pad) / s.stride; if (q_hi > s.Q - 1) q_hi = s.Q - 1;
        for (int p = p_lo; p <= p_hi; ++p) {
            const int h0 = p * s.stride - s.pad;
            for (int q = q_lo; q <= q_hi; ++q) {
                const int w0 = q * s.stride - s.pad;
                bool first_max = true;
                for (int rr = 0; rr < s.R && first_max; ++rr) {
                    const int ih = h0 + rr;
                    if (ih < 0 || ih >= s.H) continue;
                    for (int ss = 0; ss < s.R; ++ss) {
                        const int iw = w0 + ss;
                        if (iw < 0 || iw >= s.W) continue;
                        const float v = __ldg(&x[(((int64_t)n * s.H + ih) * s.W + iw) * s.C + c]);
                        const bool before = (ih < h) || (ih == h && iw < w);
                        if (v > mine || (before && v == mine)) { first_max = false; break; }
                    }
                }
                if (first_max) acc += __ldg(&dy[(((int64_t)n * s.P + p) * s.Q + q) * s.C + c]);
            }
        }
        dx[i] = ACCUM ? dx[i] + acc : acc;
    }
}

// The same routing, four channels per thread (C a multiple of 4): a quarter of the load instructions.
template <bool ACCUM>
__global__ void __launch_bounds__(kThreads)
maxpool_bwd_vec4_kernel(const float4* __restrict__ x, const float4* __restrict__ dy, float4* __restrict__ dx, ConvShape s)
{
    const int C4 = s.C / 4;
    const int64_t total = (int64_t)s.N * s.H * s.W * C4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c = (int)(i % C4);
        int64_t r = i / C4;
        const int w = (int)(r % s.W); r /= s.W;
        const int h = (int)(r % s.H);
        const int n = (int)(r / s.H);
        const float4 mine = __ldg(&x[i]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        int p_lo = h + s.pad - s.R + 1; p_lo = p_lo <= 0 ? 0 : (p_lo + s.stride - 1) / s.stride;
        int p_hi = (h + s.pad) / s.stride; if (p_hi > s.P - 1) p_hi = s.P - 1;
        int q_lo = w + s.pad - s.R + 1; q_lo = q_lo <= 0 ? 0 : (q_lo + s.stride - 1) / s.stride;
        int q_hi = (w + s.pad) / s.stride; if (q_hi > s.Q - 1) q_hi = s.Q - 1;
        for (int p = p_lo; p <= p_hi; ++p) {
            const int h0 = p * s.stride - s.pad;
            for (int q = q_lo; q <= q_hi; ++q) {
                const int w0 = q * s.stride - s.pad;
                bool f0 = true, f1 = true, f2 = true, f3 = true;          // still the first maximum of this window
                for (int rr = 0; rr < s.R; ++rr) {
                    const int ih = h0 + rr;
                    if (ih < 0 || ih >= s.H) continue;
                    for (int ss = 0; ss < s.R; ++ss) {
                        const int iw = w0 + ss;
                        if (iw < 0 || iw >= s.W) continue;
                        const float4 v = __ldg(&x[(((int64_t)n * s.H + ih) * s.W + iw) * C4 + c]);
                        const bool before = (ih < h) || (ih == h && iw < w);
                        f0 = f0 && !(v.x > mine.x || (before && v.x == mine.x));
                        f1 = f1 && !(v.y > mine.y || (before && v.y == mine.y));
                        f2 = f2 && !(v.z > mine.z || (before && v.z == mine.z));
                        f3 = f3 && !(v.w > mine.w || (before && v.w == mine.w));
                    }
                }
                if (f0 || f1 || f2 || f3) {
                    const float4 g = __ldg(&dy[(((int64_t)n * s.P + p) * s.Q + q) * C4 + c]);
                    if (f0) acc.x += g.x;
                    if (f1) acc.y += g.y;
                    if (f2) acc.z += g.z;
                    if (f3) acc.w += g.w;
                }
            }
        }
        if (ACCUM) { const float4 e = dx[i]; acc.x += e.x; acc.y += e.y; acc.z += e.z; acc.w += e.w; }
        dx[i] = acc;
    }
}

// ------------------------------------------------------------------------------------------------
// head: global average pool + FC + softmax cross-entropy
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ float block_reduce(float v, bool is_max, float* sh)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    float r = sh[0];
    for (int k = 1; k < (int)(blockDim.x >> 5); ++k) r = is_max ? fmaxf(r, sh[k]) : r + sh[k];
    return r;
}

// one block per sample; dynamic smem: C + ncls floats
__global__ void __launch_bounds__(kThreads)
head_fwd_kernel(const float* __restrict__ a, const float* __restrict__ Wfc, const float* __restrict__ bias,
                const int32_t* __restrict__ labels, float* __restrict__ logits, float* __restrict__ pooled,
                float* __restrict__ persample, int HW, int C, int ncls)
{
    extern __shared__ float smem[];
    __shared__ float red[32];
    float* sp = smem;            // pooled [C]
    float* sl = smem + C;        // logits [ncls]
    const int n = blockIdx.x, t = threadIdx.x;
    const float inv = 1.f / (float)HW;
    for (int c = t; c < C; c += blockDim.x) {
        float s = 0.f;
        for (int i = 0; i < HW; ++i) s += __ldg(&a[((int64_t)n * HW + i) * C + c]);
        const float pv = s * inv;
        sp[c] = pv;
        pooled[(int64_t)n * C + c] = pv;
    }
    __syncthreads();
    const int lane = t & 31, wid = t >> 5, nw = blockDim.x >> 5;
    for (int j = wid; j < ncls; j += nw) {
        float s = 0.f;
        for (int c = lane; c < C; c += 32) s = fmaf(sp[c], __ldg(&Wfc[(int64_t)j * C + c]), s);
        s = warp_sum(s);
        if (lane == 0) { const float lg = s + __ldg(&bias[j]); sl[j] = lg; logits[(int64_t)n * ncls + j] = lg; }
    }
    __syncthreads();
    float mx = -INFINITY;
    for (int j = t; j < ncls; j += blockDim.x) mx = fmaxf(mx, sl[j]);
    mx = block_reduce(mx, true, red);
    float z = 0.f;
    for (int j = t; j < ncls; j += blockDim.x) z += expf(sl[j] - mx);
    z = block_reduce(z, false, red);
    if (t == 0) persample[n] = -(sl[labels[n]] - mx - logf(z));
}

__global__ void head_loss_kernel(const float* __restrict__ persample, float* __restrict__ loss_slot, int b)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        float s = 0.f;
        for (int n = 0; n < b; ++n) s += persample[n];
        *loss_slot = s / (float)b;
    }
}

// one block per sample: dlogits = (softmax - onehot)/b, da[n,i,c] = (dlogits . W[:,c]) / HW
__global__ void __launch_bounds__(kThreads)
head_bwd_data_kernel(const float* __restrict__ Wfc, const int32_t* __restrict__ labels, const float* __restrict__ logits,
                     float* __restrict__ dlogits, float* __restrict__ da, int b, int HW, int C, int ncls)
{
    extern __shared__ float smem[];
    __shared__ float red[32];
    float* sd = smem;            // dlogits [ncls]
    const int n = blockIdx.x, t = threadIdx.x;
    float mx = -INFINITY;
    for (int j = t; j < ncls; j += blockDim.x) mx = fmaxf(mx, __ldg(&logits[(int64_t)n * ncls + j]));
    mx = block_reduce(mx, true, red);
    float z = 0.f;
    for (int j = t; j < ncls; j += blockDim.x) z += expf(__ldg(&logits[(int64_t)n * ncls + j]) - mx);
    z = block_reduce(z, false, red);
    const int lab = labels[n];
    const float invb = 1.f / (float)b;
    for (int j = t; j < ncls; j += blockDim.x) {
        const float p = expf(__ldg(&logits[(int64_t)n * ncls + j]) - mx) / z;
        const float d = (p - (j == lab ? 1.f : 0.f)) * invb;
        sd[j] = d;
        dlogits[(int64_t)n * ncls + j] = d;
    }
    __syncthreads();
    const float inv = 1.f / (float)HW;
    for (int c = t; c < C; c += blockDim.x) {
        float s = 0.f;
        for (int j = 0; j < ncls; ++j) s = fmaf(sd[j], __ldg(&Wfc[(int64_t)j * C + c]), s);
        s *= inv;
        for (int i = 0; i < HW; ++i) da[((int64_t)n * HW + i) * C + c] = s;
    }
}

// one block per class: dW[j][c] = sum_n dlogits[n][j] * pooled[n][c] (ascending n), dbias[j] = sum_n dlogits[n][j]
__global__ void __launch_bounds__(kThreads)
head_bwd_param_kernel(const float* __restrict__ dlogits, const float* __restrict__ pooled, float* __restrict__ dW,
                      float* __restrict__ dbias, int b, int C, int ncls)
{
    const int j = blockIdx.x, t = threadIdx.x;
    for (int c = t; c < C; c += blockDim.x) {
        float s = 0.f;
        for (int n = 0; n < b; ++n) s = fmaf(__ldg(&dlogits[(int64_t)n * ncls + j]), __ldg(&pooled[(int64_t)n * C + c]), s);
        dW[(int64_t)j * C + c] = s;
    }
    if (t == 0) {
        float s = 0.f;
        for (int n = 0; n < b; ++n) s += dlogits[(int64_t)n * ncls + j];
        dbias[j] = s;
    }
}

// ---- wide heads (ImageNet layout: 2048 channels x 1000 classes): the same arithmetic spread over the GPU ----
// pooled[n][c] = mean over the map; grid (ceil(C/256), b)
__global__ void __launch_bounds__(kThreads)
head_pool_kernel(const float* __restrict__ a, float* __restrict__ pooled, int HW, int C)
{
    const int c = blockIdx.x * kThreads + threadIdx.x, n = blockIdx.y;
    if (c >= C) return;
    float s = 0.f;
    for (int i = 0; i < HW; ++i) s += __ldg(&a[((int64_t)n * HW + i) * C + c]);
    pooled[(int64_t)n * C + c] = s * (1.f / (float)HW);
}

// logits[n][j] = pooled[n] . W[j] + bias[j]: one warp per class (a row of W is read once for eight samples at a time)
__global__ void __launch_bounds__(kThreads)
head_logits_kernel(const float* __restrict__ pooled, const float* __restrict__ Wfc, const float* __restrict__ bias,
                   float* __restrict__ logits, int b, int C, int ncls)
{
    const int lane = threadIdx.x & 31, j = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (j >= ncls) return;
    for (int n0 = 0; n0 < b; n0 += 8) {
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] = 0.f;
        for (int c = lane; c < C; c += 32) {
            const float w = __ldg(&Wfc[(int64_t)j * C + c]);
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (n0 + q < b) acc[q] = fmaf(pooled[(int64_t)(n0 + q) * C + c], w, acc[q]);
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float sum = warp_sum(acc[q]);
            if (lane == 0 && n0 + q < b) logits[(int64_t)(n0 + q) * ncls + j] = sum + __ldg(&bias[j]);
        }
    }
}

// per-sample loss from the logits; one block per sample
__global__ void __launch_bounds__(kThreads)
head_softmax_loss_kernel(const float* __restrict__ logits, const int32_t* __restrict__ labels, float* __restrict__ persample, int ncls)
{
    __shared__ float red[32];
    const int n = blockIdx.x, t = threadIdx.x;
    const float* lg = logits + (int64_t)n * ncls;
    float mx = -INFINITY;
    for (int j = t; j < ncls; j += blockDim.x) mx = fmaxf(mx, lg[j]);
    mx = block_reduce(mx, true, red);
    float z = 0.f;
    for (int j = t; j < ncls; j += blockDim.x) z += expf(lg[j] - mx);
    z = block_reduce(z, false, red);
    if (t == 0) persample[n] = -(lg[labels[n]] - mx - logf(z));
}

// dlogits = (softmax - onehot) / b; one block per sample
__global__ void __launch_bounds__(kThreads)
head_dlogits_kernel(const int32_t* __restrict__ labels, const float* __restrict__ logits, float* __restrict__ dlogits, int b, int ncls)
{
    __shared__ float red[32];
    const int n = blockIdx.x, t = threadIdx.x;
    const float* lg = logits + (int64_t)n * ncls;
    float mx = -INFINITY;
    for (int j = t; j < ncls; j += blockDim.x) mx = fmaxf(mx, __ldg(&lg[j]));
    mx = block_reduce(mx, true, red);
    float z = 0.f;
    for (int j = t; j < ncls; j += blockDim.x) z += expf(__ldg(&lg[j]) - mx);
    z = block_reduce(z, false, red);
    const int lab = labels[n];
    const float invb = 1.f / (float)b;
    for (int j = t; j < ncls; j += blockDim.x) {
        const float p = expf(__ldg(&lg[j]) - mx) / z;
        dlogits[(int64_t)n * ncls + j] = (p - (j == lab ? 1.f : 0.f)) * invb;
    }
}

// da[n][i][c] = (dlogits[n] . W[:, c]) / HW for every pixel i.  A block owns 64 channels and 8 samples; its 256 threads are
// 64 channels x 4 interleaved class slices (added in slice order).  grid (ceil(C/64), ceil(b/8)); dynamic smem 8*ncls floats.
__global__ void __launch_bounds__(kThreads)
head_bwd_pool_kernel(const float* __restrict__ Wfc, const float* __restrict__ dlogits, float* __restrict__ da, int b, int HW,
                     int C, int ncls)
{
    extern __shared__ float sd[];                      // [8][ncls]
    __shared__ float red[4][8][64];
    __shared__ float res[8][64];
    const int t = threadIdx.x, cl = t & 63, js = t >> 6;
    const int c0 = blockIdx.x * 64, n0 = blockIdx.y * 8;
    for (int idx = t; idx < 8 * ncls; idx += kThreads) {
        const int q = idx / ncls, j = idx - q * ncls;
        sd[idx] = n0 + q < b ? __ldg(&dlogits[(int64_t)(n0 + q) * ncls + j]) : 0.f;
    }
    __syncthreads();
    float acc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc[q] = 0.f;
    const int c = c0 + cl;
    if (c < C) {
#pragma unroll 4
        for (int j = js; j < ncls; j += 4) {
            const float w = __ldg(&Wfc[(int64_t)j * C + c]);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[q] = fmaf(sd[q * ncls + j], w, acc[q]);
        }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) red[js][q][cl] = acc[q];
    __syncthreads();
    const float inv = 1.f / (float)HW;
    for (int o = t; o < 8 * 64; o += kThreads) {
        const int q = o >> 6, k = o & 63;
        res[q][k] = (((red[0][q][k] + red[1][q][k]) + red[2][q][k]) + red[3][q][k]) * inv;
    }
    __syncthreads();
    const int total = 8 * HW * 64;
    for (int idx = t; idx < total; idx += kThreads) {
        const int k = idx & 63, rest = idx >> 6;
        const int i = rest % HW, q = rest / HW;
        if (n0 + q < b && c0 + k < C) da[((int64_t)(n0 + q) * HW + i) * C + c0 + k] = res[q][k];
    }
}

inline bool head_is_wide(int C, int ncls) { return ncls >= 64 && (int64_t)C * ncls >= 32768; }   // one warp per class: needs many classes

inline void count(int64_t* n_launch, int k) { if (n_launch) *n_launch += k; }

}  // namespace

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
size_t bn_scratch_bytes(int64_t rows, int C)
{
    const BnPlan p = bn_plan(rows, C);
    return 256 + ((size_t)p.nblk * 2 * C + 2 * (size_t)C) * sizeof(float);
}

// The large-tensor apply kernels keep up to 2048 channels of coefficients in dynamic shared memory beyond the default limit.
// The attribute is set once per device; if that fails the callers stay on the ticket path, which needs none.
bool big_apply_attributes_set()
{
    static signed char state[64];        // 0 not tried, 1 set, -1 failed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return false; }
    if (state[dev] == 0) {
        const int mx = (int)bn_big_apply_smem(2048);
        bool ok = cudaFuncSetAttribute(bn_apply_big_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, mx) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(bn_apply_big_bwd_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(bn_apply_big_bwd_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(bn_apply_big_bwd_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(bn_apply_big_bwd_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx) == cudaSuccess;
        if (!ok) (void)cudaGetLastError();
        state[dev] = ok ? 1 : -1;
    }
    return state[dev] == 1;
}

cudaError_t bnrelu_fwd(const float* x, const float* gamma, const float* beta, float eps, float* y, float* stats,
                       int64_t rows, int C, void* scratch, cudaStream_t st, int64_t* n_launch, bool relu)
{
    const BnPlan p = bn_plan(rows, C);
    const float floor = relu ? 0.f : -INFINITY;
    unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch);
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + 256);
    const BnClusterPlan cp = g_bn_cluster ? bn_cluster_plan(rows, C) : BnClusterPlan{false, 0, 0, 0, 0};
    if (cp.ok) {
        const float4* x4 = reinterpret_cast<const float4*>(x);
        float4* y4 = reinterpret_cast<float4*>(y);
        const int grid = cp.n_clusters * kBnCluster;
        cudaError_t e;
        if (cp.nv == 1) e = launch_cluster_pdl(bn_fwd_cluster_kernel<1>, grid, kBnThreads, kBnCluster, st, x4, gamma, beta, eps, y4, stats, rows, C, cp.cgc, cp.rows_per_cta, floor);
        else if (cp.nv == 2) e = launch_cluster_pdl(bn_fwd_cluster_kernel<2>, grid, kBnThreads, kBnCluster, st, x4, gamma, beta, eps, y4, stats, rows, C, cp.cgc, cp.rows_per_cta, floor);
        else if (cp.nv == 4) e = launch_cluster_pdl(bn_fwd_cluster_kernel<4>, grid, kBnThreads, kBnCluster, st, x4, gamma, beta, eps, y4, stats, rows, C, cp.cgc, cp.rows_per_cta, floor);
        else e = launch_cluster_pdl(bn_fwd_cluster_kernel<8>, grid, kBnThreads, kBnCluster, st, x4, gamma, beta, eps, y4, stats, rows, C, cp.cgc, cp.rows_per_cta, floor);
        count(n_launch, 1);
        return e;
    }
    const BnBigPlan bp = bn_big_plan<false>(rows, C, p);
    if (bp.ok && big_apply_attributes_set()) {
        const size_t smem = bn_big_apply_smem(C);
        launch_cluster_pdl(bn_reduce_big_kernel<false>, bp.n_clusters * kBnBigCluster, kBnThreads, kBnBigCluster, st,
                           reinterpret_cast<const float4*>(x), (const float4*)nullptr, gamma, beta, (const float*)nullptr, rows, C,
                           p.cgt, p.rl, bp.rows_per_blk, partials, floor);
        launch_pdl(bn_apply_big_fwd_kernel, bp.nblk_apply, kBnThreads, smem, st, reinterpret_cast<const float4*>(x), gamma, beta,
                   (const float*)partials, bp.n_clusters, eps, stats, reinterpret_cast<float4*>(y), rows, C, p.cgt, p.rl,
                   bp.rows_per_blk_apply, floor, bp.stream_out);
        count(n_launch, 2);
        return cudaGetLastError();
    }
    launch_pdl(bn_reduce_kernel<false>, p.nblk, kBnThreads, 0, st, x, (const float*)nullptr, gamma, beta, (const float*)nullptr, eps, rows, C, p.cgt, p.rl,
                                                           p.passes, p.rows_per_blk, ticket, partials, stats, stats + C,
                                                           (float*)nullptr, floor);
    launch_pdl(bn_apply_fwd_kernel, p.nblk_apply, kBnThreads, 0, st, reinterpret_cast<const float4*>(x), gamma, beta, stats,
                                                             reinterpret_cast<float4*>(y), rows, C, p.cgt, p.rl, p.passes,
                                                             p.rows_per_blk_apply, floor);
    count(n_launch, 2);
    return cudaGetLastError();
}

cudaError_t bnrelu_bwd(const float* x, const float* dy, const float* gamma, const float* beta, const float* stats,
                       float* dx, const float* addend, bool accumulate, float* dgamma, float* dbeta, int64_t rows,
                       int C, void* scratch, cudaStream_t st, int64_t* n_launch, bool relu, bool x_is_old)
{
    const BnPlan p = bn_plan(rows, C);
    const float floor = relu ? 0.f : -INFINITY;
    const BnClusterPlan cp = g_bn_cluster ? bn_cluster_plan(rows, C) : BnClusterPlan{false, 0, 0, 0, 0};
    if (cp.ok) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(cp.n_clusters * kBnCluster); cfg.blockDim = dim3(kBnThreads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kBnCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = g_pdl_enabled ? 2 : 1;
        const float4* x4 = reinterpret_cast<const float4*>(x);
        const float4* dy4 = reinterpret_cast<const float4*>(dy);
        const float4* ad4 = reinterpret_cast<const float4*>(addend);
        float4* dx4 = reinterpret_cast<float4*>(dx);
        const int early = x_is_old ? 1 : 0;
        cudaError_t e;
#define HPF_BN_CL(NV, A, B) e = cudaLaunchKernelEx(&cfg, bn_bwd_cluster_kernel<NV, A, B>, x4, dy4, gamma, beta, stats, ad4, dx4, dgamma, dbeta, rows, C, cp.cgc, cp.rows_per_cta, floor, early)
#define HPF_BN_CL_NV(NV) do { if (addend && accumulate) HPF_BN_CL(NV, true, true); else if (addend) HPF_BN_CL(NV, true, false); \
                              else if (accumulate) HPF_BN_CL(NV, false, true); else HPF_BN_CL(NV, false, false); } while (0)
        if (cp.nv == 1) HPF_BN_CL_NV(1); else if (cp.nv == 2) HPF_BN_CL_NV(2); else if (cp.nv == 4) HPF_BN_CL_NV(4); else HPF_BN_CL_NV(8);
#undef HPF_BN_CL_NV
#undef HPF_BN_CL
        count(n_launch, 1);
        return e;
    }
    unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch);
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + 256);
    float* coef = partials + (size_t)p.nblk * 2 * C;
    const BnBigPlan bp = bn_big_plan<true>(rows, C, p);
    if (bp.ok && big_apply_attributes_set()) {
        const size_t smem = bn_big_apply_smem(C);
        const float4* x4 = reinterpret_cast<const float4*>(x);
        const float4* dy4 = reinterpret_cast<const float4*>(dy);
        const float4* ad4 = reinterpret_cast<const float4*>(addend);
        float4* dx4 = reinterpret_cast<float4*>(dx);
        launch_cluster_pdl(bn_reduce_big_kernel<true>, bp.n_clusters * kBnBigCluster, kBnThreads, kBnBigCluster, st, x4, dy4, gamma, beta,
                           stats, rows, C, p.cgt, p.rl, bp.rows_per_blk, partials, floor);
#define HPF_BN_BIG(A, B) launch_pdl(bn_apply_big_bwd_kernel<A, B>, bp.nblk_apply, kBnThreads, smem, st, x4, dy4, gamma, beta, stats, (const float*)partials, bp.n_clusters, dgamma, dbeta, ad4, dx4, rows, C, p.cgt, p.rl, bp.rows_per_blk_apply, floor, bp.stream_out)
        if (addend && accumulate) HPF_BN_BIG(true, true);
        else if (addend) HPF_BN_BIG(true, false);
        else if (accumulate) HPF_BN_BIG(false, true);
        else HPF_BN_BIG(false, false);
#undef HPF_BN_BIG
        count(n_launch, 2);
        return cudaGetLastError();
    }
    launch_pdl(bn_reduce_kernel<true>, p.nblk, kBnThreads, 0, st, x, dy, gamma, beta, stats, 0.f, rows, C, p.cgt, p.rl, p.passes,
                                                          p.rows_per_blk, ticket, partials, dbeta, dgamma, coef, floor);
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const float4* dy4 = reinterpret_cast<const float4*>(dy);
    const float4* ad4 = reinterpret_cast<const float4*>(addend);
    float4* dx4 = reinterpret_cast<float4*>(dx);
    const int nb = p.nblk_apply;
#define HPF_BN_APPLY(A, B) launch_pdl(bn_apply_bwd_kernel<A, B>, nb, kBnThreads, 0, st, x4, dy4, gamma, beta, stats, coef, ad4, dx4, rows, C, p.cgt, p.rl, p.passes, p.rows_per_blk_apply, floor)
    if (addend && accumulate) HPF_BN_APPLY(true, true);
    else if (addend) HPF_BN_APPLY(true, false);
    else if (accumulate) HPF_BN_APPLY(false, true);
    else HPF_BN_APPLY(false, false);
#undef HPF_BN_APPLY
    count(n_launch, 2);
    return cudaGetLastError();
}

cudaError_t bnrelu_fwd_apply(const float* x, const float* gamma, const float* beta, const float* stats, float* y,
                             int64_t rows, int C, cudaStream_t st, int64_t* n_launch)
{
    const BnPlan p = bn_plan(rows, C);
    launch_pdl(bn_apply_fwd_kernel, p.nblk_apply, kBnThreads, 0, st, reinterpret_cast<const float4*>(x), gamma, beta, stats,
               reinterpret_cast<float4*>(y), rows, C, p.cgt, p.rl, p.passes, p.rows_per_blk_apply, 0.f);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t relu_fwd(const float* x, float* y, int64_t n, cudaStream_t st, int64_t* n_launch)
{
    launch_pdl(relu_fwd_kernel, ew_blocks(n / 4 + 1), kThreads, 0, st, x, y, n);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t relu_bwd(const float* x, const float* dy, float* dx, const float* addend, bool accumulate, int64_t n, cudaStream_t st,
                     int64_t* n_launch)
{
    const int nb = ew_blocks(n / 4 + 1);
    if (addend && accumulate) launch_pdl(relu_bwd_kernel<true, true>, nb, kThreads, 0, st, x, dy, addend, dx, n);
    else if (addend) launch_pdl(relu_bwd_kernel<true, false>, nb, kThreads, 0, st, x, dy, addend, dx, n);
    else if (accumulate) launch_pdl(relu_bwd_kernel<false, true>, nb, kThreads, 0, st, x, dy, addend, dx, n);
    else launch_pdl(relu_bwd_kernel<false, false>, nb, kThreads, 0, st, x, dy, addend, dx, n);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t add_fwd(const float* a, const float* b, float* out, int64_t n, cudaStream_t st, int64_t* n_launch)
{
    launch_pdl(add_kernel, ew_blocks(n / 4 + 1), kThreads, 0, st, a, b, out, n);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t grad_accumulate(float* dst, const float* src, int64_t n, bool accumulate, cudaStream_t st, int64_t* n_launch)
{
    if (accumulate) launch_pdl(accumulate_kernel<true>, ew_blocks(n / 4 + 1), kThreads, 0, st, dst, src, n);
    else launch_pdl(accumulate_kernel<false>, ew_blocks(n / 4 + 1), kThreads, 0, st, dst, src, n);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t grad_average(const float* slots, float* out, int M, int64_t G, cudaStream_t st, int64_t* n_launch)
{
    const float inv_m = 1.f / (float)M;
    const bool out16 = (reinterpret_cast<uintptr_t>(out) & 15u) == 0 && (reinterpret_cast<uintptr_t>(slots) & 15u) == 0;
    if (G % 4 == 0 && out16) grad_average_kernel<4><<<ew_blocks(G / 4), kThreads, 0, st>>>(slots, out, M, G, inv_m);
    else if (G % 2 == 0 && out16) grad_average_kernel<2><<<ew_blocks(G / 2), kThreads, 0, st>>>(slots, out, M, G, inv_m);
    else grad_average_kernel<1><<<ew_blocks(G), kThreads, 0, st>>>(slots, out, M, G, inv_m);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t sgd_momentum(const float* slots, float* gavg, float* theta, float* vel, int M, int64_t G, float lr, float mu,
                         float wd, cudaStream_t st, int64_t* n_launch)
{
    const float inv_m = 1.f / (float)M;
    const uintptr_t all = reinterpret_cast<uintptr_t>(slots) | reinterpret_cast<uintptr_t>(gavg) | reinterpret_cast<uintptr_t>(theta) |
                          reinterpret_cast<uintptr_t>(vel);
    if (G % 4 == 0 && (all & 15u) == 0) sgd_momentum_kernel<4><<<ew_blocks(G / 4), kThreads, 0, st>>>(slots, gavg, theta, vel, M, G, inv_m, lr, mu, wd);
    else sgd_momentum_kernel<1><<<ew_blocks(G), kThreads, 0, st>>>(slots, gavg, theta, vel, M, G, inv_m, lr, mu, wd);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t stamp_time(unsigned long long* slot, cudaStream_t st, int64_t* n_launch)
{
    stamp_kernel<<<1, 1, 0, st>>>(slot);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t loss_average(const float* loss_slots, float* out, int M, cudaStream_t st, int64_t* n_launch)
{
    loss_average_kernel<<<1, 32, 0, st>>>(loss_slots, out, M);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t maxpool_fwd(const float* x, float* y, ConvShape s, cudaStream_t st, int64_t* n_launch)
{
    maxpool_fwd_kernel<<<ew_blocks((int64_t)s.N * s.P * s.Q * s.C), kThreads, 0, st>>>(x, y, s);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t maxpool_bwd(const float* x, const float* dy, float* dx, bool accumulate, ConvShape s, cudaStream_t st,
                        int64_t* n_launch)
{
    const bool vec4 = s.C % 4 == 0 && ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(dy) | reinterpret_cast<uintptr_t>(dx)) & 15u) == 0;
    if (vec4) {
        const int nb = ew_blocks((int64_t)s.N * s.H * s.W * (s.C / 4));
        const float4* x4 = reinterpret_cast<const float4*>(x);
        const float4* dy4 = reinterpret_cast<const float4*>(dy);
        float4* dx4 = reinterpret_cast<float4*>(dx);
        if (accumulate) maxpool_bwd_vec4_kernel<true><<<nb, kThreads, 0, st>>>(x4, dy4, dx4, s);
        else maxpool_bwd_vec4_kernel<false><<<nb, kThreads, 0, st>>>(x4, dy4, dx4, s);
        count(n_launch, 1);
        return cudaGetLastError();
    }
    const int nb = ew_blocks((int64_t)s.N * s.H * s.W * s.C);
    if (accumulate) maxpool_bwd_kernel<true><<<nb, kThreads, 0, st>>>(x, dy, dx, s);
    else maxpool_bwd_kernel<false><<<nb, kThreads, 0, st>>>(x, dy, dx, s);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t head_fwd(const float* a, const float* Wfc, const float* bias, const int32_t* labels, float* logits,
                     float* pooled, float* persample, float* loss_slot, int b, int HW, int C, int ncls,
                     cudaStream_t st, int64_t* n_launch)
{
    if (head_is_wide(C, ncls)) {
        head_pool_kernel<<<dim3((C + kThreads - 1) / kThreads, b), kThreads, 0, st>>>(a, pooled, HW, C);
        head_logits_kernel<<<(ncls + kThreads / 32 - 1) / (kThreads / 32), kThreads, 0, st>>>(pooled, Wfc, bias, logits, b, C, ncls);
        head_softmax_loss_kernel<<<b, kThreads, 0, st>>>(logits, labels, persample, ncls);
        head_loss_kernel<<<1, 32, 0, st>>>(persample, loss_slot, b);
        count(n_launch, 4);
        return cudaGetLastError();
    }
    const size_t smem = (size_t)(C + ncls) * sizeof(float);
    head_fwd_kernel<<<b, kThreads, smem, st>>>(a, Wfc, bias, labels, logits, pooled, persample, HW, C, ncls);
    head_loss_kernel<<<1, 32, 0, st>>>(persample, loss_slot, b);
    count(n_launch, 2);
    return cudaGetLastError();
}

cudaError_t head_bwd(const float* Wfc, const int32_t* labels, const float* logits, const float* pooled,
                     float* dlogits, float* da, float* dW, float* dbias, int b, int HW, int C, int ncls,
                     cudaStream_t st, int64_t* n_launch)
{
    if (head_is_wide(C, ncls) && (size_t)8 * ncls * sizeof(float) <= 40 * 1024) {
        head_dlogits_kernel<<<b, kThreads, 0, st>>>(labels, logits, dlogits, b, ncls);
        head_bwd_pool_kernel<<<dim3((C + 63) / 64, (b + 7) / 8), kThreads, (size_t)8 * ncls * sizeof(float), st>>>(Wfc, dlogits, da, b, HW, C, ncls);
        head_bwd_param_kernel<<<ncls, kThreads, 0, st>>>(dlogits, pooled, dW, dbias, b, C, ncls);
        count(n_launch, 3);
        return cudaGetLastError();
    }
    head_bwd_data_kernel<<<b, kThreads, (size_t)ncls * sizeof(float), st>>>(Wfc, labels, logits, dlogits, da, b, HW, C, ncls);
    head_bwd_param_kernel<<<ncls, kThreads, 0, st>>>(dlogits, pooled, dW, dbias, b, C, ncls);
    count(n_launch, 2);
    return cudaGetLastError();
}

}  // namespace hpf
