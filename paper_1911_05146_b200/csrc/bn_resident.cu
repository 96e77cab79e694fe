// BN(training)+ReLU forward with the whole tensor held on chip between the statistics and the apply step.
//
// Batch normalisation needs the statistics of the whole tensor before its first output element, so a two-kernel
// scheme reads the input twice.  A tensor of up to a few tens of MB fits the registers and the shared memory of
// all SMs together (148 x (96 KB of registers + 176 KB of shared memory)): one cooperative launch of one CTA per SM
// reads its share of x once, keeps it, exchanges per-channel partial sums through a small global buffer and a
// grid-wide barrier, and writes y from the held copy.  HBM traffic is the algorithmic 8 bytes per element.
//
// The launch occupies every SM until its slowest CTA has passed the barrier, so it is meant for a call that has
// the GPU to itself (the single-op entry point); the pipelined step keeps its own kernels.
#include "hpf_kernels.h"

#include <math.h>
#include <stdlib.h>

namespace hpf {

namespace {

// -DHPF_RES_TIMELINE: thread 0 of every CTA stamps the nanosecond timer at the phase boundaries of the forward kernel
// into the scratch behind the partial rows (8 stamps per CTA), for latency studies.
#ifdef HPF_RES_TIMELINE
#define RES_STAMP(k) do { if (threadIdx.x == 0) tl[blockIdx.x * 8 + (k)] = res_timer(); } while (0)
#else
#define RES_STAMP(k) do { } while (0)
#endif

constexpr int kResThreads = 1024;
constexpr int kResRegV = 6;                       // float4 per thread kept in registers
constexpr int kResSmemV = 11;                     // float4 per thread kept in shared memory, at most
constexpr unsigned long long kResWaitNs = 2000000000ull;   // the barrier gives up after two seconds

__device__ __forceinline__ float res_xhat(float x, float mean, float rstd) { return (x - mean) * rstd; }
__device__ __forceinline__ float res_z(float xh, float g, float b) { return fmaf(g, xh, b); }

__device__ __forceinline__ unsigned long long res_timer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned int res_ld_acquire(const unsigned int* p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void res_cp_async16(void* smem_dst, const void* gsrc)
{
    const unsigned int d = (unsigned int)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void res_cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void res_acc(float4& a, float4& b, const float4& v, const float4& sh)
{
    float d;
    d = v.x - sh.x; a.x += d; b.x = fmaf(d, d, b.x);
    d = v.y - sh.y; a.y += d; b.y = fmaf(d, d, b.y);
    d = v.z - sh.z; a.z += d; b.z = fmaf(d, d, b.z);
    d = v.w - sh.w; a.w += d; b.w = fmaf(d, d, b.w);
}
__device__ __forceinline__ float4 res_apply(const float4& v, const float4& mu, const float4& rs, const float4& g, const float4& bt,
                                            float floor)
{
    float4 o;
    o.x = fmaxf(res_z(res_xhat(v.x, mu.x, rs.x), g.x, bt.x), floor);
    o.y = fmaxf(res_z(res_xhat(v.y, mu.y, rs.y), g.y, bt.y), floor);
    o.z = fmaxf(res_z(res_xhat(v.z, mu.z, rs.z), g.z, bt.z), floor);
    o.w = fmaxf(res_z(res_xhat(v.w, mu.w, rs.w), g.w, bt.w), floor);
    return o;
}

constexpr int kResRegBwd = 4;                     // backward, dz only: float4 per thread in registers
constexpr int kResRegBwdBoth = 2;                 // backward, dz and xhat: pairs per thread in registers
__device__ __forceinline__ float4 res_xhat4(const float4& v, const float4& mu, const float4& rs)
{
    return make_float4(res_xhat(v.x, mu.x, rs.x), res_xhat(v.y, mu.y, rs.y), res_xhat(v.z, mu.z, rs.z), res_xhat(v.w, mu.w, rs.w));
}
__device__ __forceinline__ void res_dz(const float4& v, const float4& d, const float4& mu, const float4& rs, const float4& g,
                                       const float4& bt, float floor, float4& xh, float4& dz)
{
    xh = res_xhat4(v, mu, rs);
    dz.x = res_z(xh.x, g.x, bt.x) > floor ? d.x : 0.f;
    dz.y = res_z(xh.y, g.y, bt.y) > floor ? d.y : 0.f;
    dz.z = res_z(xh.z, g.z, bt.z) > floor ? d.z : 0.f;
    dz.w = res_z(xh.w, g.w, bt.w) > floor ? d.w : 0.f;
}
__device__ __forceinline__ void res_acc_bwd(float4& a, float4& b, const float4& dz, const float4& xh)
{
    a.x += dz.x; b.x = fmaf(dz.x, xh.x, b.x);
    a.y += dz.y; b.y = fmaf(dz.y, xh.y, b.y);
    a.z += dz.z; b.z = fmaf(dz.z, xh.z, b.z);
    a.w += dz.w; b.w = fmaf(dz.w, xh.w, b.w);
}
__device__ __forceinline__ float4 res_dx(const float4& dz, const float4& xh, const float4& sc, const float4& ca, const float4& cb)
{
    return make_float4(sc.x * (dz.x - ca.x - xh.x * cb.x), sc.y * (dz.y - ca.y - xh.y * cb.y), sc.z * (dz.z - ca.z - xh.z * cb.z),
                       sc.w * (dz.w - ca.w - xh.w * cb.w));
}

// The exchange between the two steps, the same for both directions.  Every thread brings the two sums (a, b) of its four
// channels over its elements; on return dtot[k * C4 + q] (k = 0..3: a of channel 4q+k, k = 4..7: b) holds the totals
// over the whole tensor, identical in every CTA.  False: the barrier wait gave up (sync[2] is set).
__device__ __forceinline__ bool res_exchange(float4 a, float4 b, int C4, unsigned int* sync, unsigned int gen0, float* partials,
                                             double* dred, double* dtot)
{
#ifdef HPF_RES_TIMELINE
    unsigned long long* tl = reinterpret_cast<unsigned long long*>(partials + (size_t)gridDim.x * 8 * C4);
#endif
    __shared__ int s_fail;
    float* red = reinterpret_cast<float*>(dred);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    // block reduction in a fixed order: lanes of a warp that share a channel quad first (fewer than 32 quads), then
    // over the entries of all warps
    int nent = kResThreads, e = t;
    bool writer = true;
    if (C4 < 32) {
        for (int off = 16; off >= C4; off >>= 1) {
            a.x += __shfl_xor_sync(0xffffffffu, a.x, off); a.y += __shfl_xor_sync(0xffffffffu, a.y, off);
            a.z += __shfl_xor_sync(0xffffffffu, a.z, off); a.w += __shfl_xor_sync(0xffffffffu, a.w, off);
            b.x += __shfl_xor_sync(0xffffffffu, b.x, off); b.y += __shfl_xor_sync(0xffffffffu, b.y, off);
            b.z += __shfl_xor_sync(0xffffffffu, b.z, off); b.w += __shfl_xor_sync(0xffffffffu, b.w, off);
        }
        nent = 32 * C4; e = warp * C4 + lane; writer = lane < C4;
    }
    if (writer) {
        red[0 * kResThreads + e] = a.x; red[1 * kResThreads + e] = a.y; red[2 * kResThreads + e] = a.z; red[3 * kResThreads + e] = a.w;
        red[4 * kResThreads + e] = b.x; red[5 * kResThreads + e] = b.y; red[6 * kResThreads + e] = b.z; red[7 * kResThreads + e] = b.w;
    }
    __syncthreads();
    const int nval = 8 * C4;                         // <= 1024
    if (t < nval) {
        const int k = t / C4, qq = t - k * C4;
        float s = 0.f;
#pragma unroll 8
        for (int m = qq; m < nent; m += C4) s += red[k * kResThreads + m];
        __stcg(partials + (size_t)blockIdx.x * nval + t, s);
    }

    // grid-wide barrier.  The CTA barrier orders the partial sums of all threads before thread 0's fence, which publishes
    // them ahead of the arrival.  The last CTA to arrive advances the generation at once and clears the count afterwards:
    // nobody reads the count again before the next launch.
    __syncthreads();
    RES_STAMP(6);
    if (t == 0) {
        int fail = 0;
        __threadfence();
        const unsigned int old = atomicAdd(sync, 1u);
        if (old == gridDim.x - 1) {
            __threadfence();
            atomicAdd(sync + 1, 1u);
            atomicExch(sync, 0u);
        } else {
            const unsigned long long t0 = res_timer();
            unsigned int polls = 0;
            while (res_ld_acquire(sync + 1) == gen0) {
                if ((++polls & 1023u) == 0 && res_timer() - t0 > kResWaitNs) { atomicExch(sync + 2, 1u); fail = 1; break; }
            }
        }
        s_fail = fail;
    }
    __syncthreads();
    if (s_fail) return false;
    RES_STAMP(7);

    // every CTA adds the partial rows itself: G thread groups take the rows g, g + G, ... in ascending order (fp64), then
    // the groups are added in ascending order.  A thread fetches its rows eight at a time, 128 bits each, all in flight
    // together: a loop that waited for each load in turn would pay an L2 round trip per row.
    {
        const int nv4 = nval >> 2;                   // float4 per partial row, <= 256
        int G = kResThreads / nv4;
        const int g_want = ((int)gridDim.x + 7) >> 3;
        if (G > g_want) G = g_want;
        const int g = t / nv4, v4 = t - g * nv4;
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        if (g < G) {
            const float4* prow = reinterpret_cast<const float4*>(partials) + v4;
            for (int b0 = g; b0 < (int)gridDim.x; b0 += 8 * G) {
                float4 pv[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int bI = b0 + k * G;
                    pv[k] = bI < (int)gridDim.x ? __ldcg(prow + (size_t)bI * nv4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) { s0 += (double)pv[k].x; s1 += (double)pv[k].y; s2 += (double)pv[k].z; s3 += (double)pv[k].w; }
            }
            // group sums: [g][value], value = 4 * v4 + component
            dred[g * nval + 4 * v4 + 0] = s0; dred[g * nval + 4 * v4 + 1] = s1;
            dred[g * nval + 4 * v4 + 2] = s2; dred[g * nval + 4 * v4 + 3] = s3;
        }
        __syncthreads();
        if (t < nval) {
            double tot = 0.0;
#pragma unroll 4
            for (int g2 = 0; g2 < G; ++g2) tot += dred[g2 * nval + t];
            dtot[t] = tot;
        }
        __syncthreads();
    }
    return true;
}

// sync[0]: arrival count (zero between launches), sync[1]: barrier generation, sync[2]: set when a wait gave up.
// partials: [gridDim.x][8 * C/4] floats; row layout [k][q], k = 0..3 the sums of (x - shift) of channel 4q+k,
// k = 4..7 the sums of squares.  per_cta (float4 handled by one CTA) is a multiple of C/4, so a thread's channel
// quad q = threadIdx.x % (C/4) is the same in every iteration and in every CTA.
__global__ void __launch_bounds__(kResThreads, 1)
bn_fwd_resident_kernel(const float4* __restrict__ x4, const float* __restrict__ gamma, const float* __restrict__ beta, float eps,
                       float4* __restrict__ y4, float* __restrict__ stats, long long n4, long long rows, int C, long long per_cta,
                       int iters, unsigned int* sync, float* partials, float floor)
{
    extern __shared__ float4 held[];                 // [iters - kResRegV][kResThreads]
    __shared__ double dred[4096];                    // 32 KB: float [8][1024] in the block reduction, doubles afterwards
    __shared__ double dtot[1024];                    // the 8 * C/4 totals
    __shared__ __align__(16) float s_mean[1024];     // mean [C], then rstd [C]

    const int t = threadIdx.x;
    const int C4 = C >> 2;
    const int q = t & (C4 - 1);
    const long long cta_begin = (long long)blockIdx.x * per_cta;
    long long cta_end = cta_begin + per_cta;
    if (cta_end > n4) cta_end = n4;
    const long long base = cta_begin + t;

    pdl_launch_dependents();
    pdl_wait();
#ifdef HPF_RES_TIMELINE
    unsigned long long* tl = reinterpret_cast<unsigned long long*>(partials + (size_t)gridDim.x * 8 * C4);
#endif
    RES_STAMP(0);
    unsigned int gen0 = 0;
    if (t == 0) gen0 = res_ld_acquire(sync + 1);

    // the part kept in shared memory first: asynchronous copies that need no registers
    for (int j = kResRegV; j < iters; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) res_cp_async16(&held[(j - kResRegV) * kResThreads + t], x4 + i);
    }
    const float4 sh = __ldg(x4 + q);                 // shift = row 0 (shifted sums avoid cancellation)
    const float shift_c = t < C ? __ldg(reinterpret_cast<const float*>(x4) + t) : 0.f;   // for the finalisation of channel t
    float4 r[kResRegV];
#pragma unroll
    for (int j = 0; j < kResRegV; ++j) {
        const long long i = base + (long long)j * kResThreads;
        r[j] = i < cta_end ? __ldcs(x4 + i) : sh;    // out of range: equal to the shift, adds nothing
    }
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
    for (int j = 0; j < kResRegV; ++j) res_acc(a, b, r[j], sh);
    RES_STAMP(1);
    res_cp_async_wait_all();
    RES_STAMP(2);
    for (int j = kResRegV; j < iters; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) res_acc(a, b, held[(j - kResRegV) * kResThreads + t], sh);
    }

    RES_STAMP(3);
    if (!res_exchange(a, b, C4, sync, gen0, partials, dred, dtot)) {   // no sums: poison the statistics, store no output
        if (blockIdx.x == 0) for (int c = t; c < 2 * C; c += kResThreads) stats[c] = nanf("");
        return;
    }
    float* s_rstd = s_mean + C;
    if (t < C) {
        const int qq = t >> 2, k = t & 3;
        const double inv_rows = 1.0 / (double)rows;
        const double shift = (double)shift_c;
        const double m1 = dtot[k * C4 + qq] * inv_rows;
        double var = dtot[(4 + k) * C4 + qq] * inv_rows - m1 * m1;
        if (var < 0.0) var = 0.0;
        const float mean = (float)(shift + m1);
        const float rstd = (float)(1.0 / sqrt(var + (double)eps));
        s_mean[t] = mean; s_rstd[t] = rstd;
        if (blockIdx.x == 0) { stats[t] = mean; stats[C + t] = rstd; }
    }
    __syncthreads();
    RES_STAMP(4);
    const float4 mu = reinterpret_cast<const float4*>(s_mean)[q];
    const float4 rs = reinterpret_cast<const float4*>(s_rstd)[q];
    const float4 gm = __ldg(reinterpret_cast<const float4*>(gamma) + q);
    const float4 bt = __ldg(reinterpret_cast<const float4*>(beta) + q);
#pragma unroll
    for (int j = 0; j < kResRegV; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) __stcs(y4 + i, res_apply(r[j], mu, rs, gm, bt, floor));
    }
    for (int j = kResRegV; j < iters; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) __stcs(y4 + i, res_apply(held[(j - kResRegV) * kResThreads + t], mu, rs, gm, bt, floor));
    }
    RES_STAMP(5);
}

// Backward: dz = dy * [z > floor]; a = sum dz (dbeta), b = sum dz * xhat (dgamma);
// dx = gamma * rstd * (dz - a/rows - xhat * b/rows) (+ addend) (+ dx).  What stays on chip between the two steps is dz and,
// when there is room for both (HOLD_X), xhat; otherwise x is read a second time (it was read a moment ago: L2).
// Shared-memory slots: iteration j >= NREG keeps dz in slot (j - NREG) * SL and xhat in the slot after it (HOLD_X).
template <bool HOLD_X>
__global__ void __launch_bounds__(kResThreads, 1)
bn_bwd_resident_kernel(const float4* __restrict__ x4, const float4* __restrict__ dy4, const float* __restrict__ gamma,
                       const float* __restrict__ beta, const float* __restrict__ stats, const float4* __restrict__ addend,
                       float4* __restrict__ dx4, int accumulate, float* __restrict__ dgamma, float* __restrict__ dbeta, long long n4,
                       long long rows, int C, long long per_cta, int iters, unsigned int* sync, float* partials, float floor)
{
    constexpr int NREG = HOLD_X ? kResRegBwdBoth : kResRegBwd;
    constexpr int SL = HOLD_X ? 2 : 1;
    extern __shared__ float4 held[];
    __shared__ double dred[4096];
    __shared__ double dtot[1024];
    __shared__ __align__(16) float s_coef[1024];     // a/rows [C], then b/rows [C]

    const int t = threadIdx.x;
    const int C4 = C >> 2;
    const int q = t & (C4 - 1);
    const long long cta_begin = (long long)blockIdx.x * per_cta;
    long long cta_end = cta_begin + per_cta;
    if (cta_end > n4) cta_end = n4;
    const long long base = cta_begin + t;

    pdl_launch_dependents();
    pdl_wait();
    unsigned int gen0 = 0;
    if (t == 0) gen0 = res_ld_acquire(sync + 1);

    for (int j = NREG; j < iters; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) {
            res_cp_async16(&held[((j - NREG) * SL) * kResThreads + t], dy4 + i);
            if (HOLD_X) res_cp_async16(&held[((j - NREG) * SL + 1) * kResThreads + t], x4 + i);
        }
    }
    const float4 mu = __ldg(reinterpret_cast<const float4*>(stats) + q);
    const float4 rs = __ldg(reinterpret_cast<const float4*>(stats + C) + q);
    const float4 gm = __ldg(reinterpret_cast<const float4*>(gamma) + q);
    const float4 bt = __ldg(reinterpret_cast<const float4*>(beta) + q);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    float4 rz[NREG], rx[HOLD_X ? NREG : 1];
    {
        float4 v[NREG], d[NREG];
#pragma unroll
        for (int j = 0; j < NREG; ++j) {
            const long long i = base + (long long)j * kResThreads;
            const bool in = i < cta_end;
            v[j] = in ? __ldg(x4 + i) : mu;
            d[j] = in ? __ldcs(dy4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < NREG; ++j) {
            float4 xh;
            res_dz(v[j], d[j], mu, rs, gm, bt, floor, xh, rz[j]);
            res_acc_bwd(a, b, rz[j], xh);
            if (HOLD_X) rx[j] = xh;
        }
    }
    res_cp_async_wait_all();
#pragma unroll 2
    for (int j = NREG; j < iters; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) {
            float4* slot = &held[((j - NREG) * SL) * kResThreads + t];
            const float4 d = slot[0];
            const float4 v = HOLD_X ? slot[kResThreads] : __ldg(x4 + i);
            float4 xh, dz;
            res_dz(v, d, mu, rs, gm, bt, floor, xh, dz);
            res_acc_bwd(a, b, dz, xh);
            slot[0] = dz;
            if (HOLD_X) slot[kResThreads] = xh;
        }
    }

    if (!res_exchange(a, b, C4, sync, gen0, partials, dred, dtot)) {   // no sums: poison the parameter gradients, store no dx
        if (blockIdx.x == 0) for (int c = t; c < C; c += kResThreads) { dgamma[c] = nanf(""); dbeta[c] = nanf(""); }
        return;
    }
    if (t < C) {
        const int qq = t >> 2, k = t & 3;
        const double inv_rows = 1.0 / (double)rows;
        const double sa = dtot[k * C4 + qq], sb = dtot[(4 + k) * C4 + qq];
        s_coef[t] = (float)(sa * inv_rows); s_coef[C + t] = (float)(sb * inv_rows);
        if (blockIdx.x == 0) { dbeta[t] = (float)sa; dgamma[t] = (float)sb; }
    }
    __syncthreads();
    const float4 ca = reinterpret_cast<const float4*>(s_coef)[q];
    const float4 cb = reinterpret_cast<const float4*>(s_coef + C)[q];
    float4 sc;                                       // gamma * rstd, as the two-kernel path forms it
    sc.x = gm.x * rs.x; sc.y = gm.y * rs.y; sc.z = gm.z * rs.z; sc.w = gm.w * rs.w;
#pragma unroll
    for (int j = 0; j < NREG; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) {
            float4 xh;
            if (HOLD_X) xh = rx[j];
            else { const float4 v = __ldg(x4 + i); xh = res_xhat4(v, mu, rs); }
            float4 o = res_dx(rz[j], xh, sc, ca, cb);
            if (addend) { const float4 e = __ldg(addend + i); o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            if (accumulate) { const float4 e = dx4[i]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            __stcs(dx4 + i, o);
        }
    }
#pragma unroll 2
    for (int j = NREG; j < iters; ++j) {
        const long long i = base + (long long)j * kResThreads;
        if (i < cta_end) {
            const float4* slot = &held[((j - NREG) * SL) * kResThreads + t];
            float4 xh;
            if (HOLD_X) xh = slot[kResThreads];
            else { const float4 v = __ldg(x4 + i); xh = res_xhat4(v, mu, rs); }
            float4 o = res_dx(slot[0], xh, sc, ca, cb);
            if (addend) { const float4 e = __ldg(addend + i); o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            if (accumulate) { const float4 e = dx4[i]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            __stcs(dx4 + i, o);
        }
    }
}

struct ResidentPlan { bool ok; int grid, iters; long long per_cta; size_t smem; };

// SMs of the current device if it can run these kernels (cooperative launch, one CTA per SM with the full dynamic
// shared memory); 0 otherwise.  Asked once per device.
int resident_sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cached[dev]) {
        int n = 0, coop = 0, per_sm = 0;
        const int max_dyn = kResSmemV * kResThreads * (int)sizeof(float4);
        bool ok = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
                  cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && coop != 0;
        ok = ok && cudaFuncSetAttribute(bn_fwd_resident_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(bn_bwd_resident_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(bn_bwd_resident_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn) == cudaSuccess;
        ok = ok && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bn_fwd_resident_kernel, kResThreads, max_dyn) == cudaSuccess && per_sm >= 1;
        ok = ok && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bn_bwd_resident_kernel<false>, kResThreads, max_dyn) == cudaSuccess && per_sm >= 1;
        ok = ok && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bn_bwd_resident_kernel<true>, kResThreads, max_dyn) == cudaSuccess && per_sm >= 1;
        if (!ok) { (void)cudaGetLastError(); return 0; }
        cached[dev] = n;
    }
    return cached[dev];
}

// nreg iterations of a thread stay in registers, the others take `slots` float4 of shared memory each.
ResidentPlan resident_plan(int64_t rows, int C, size_t scratch_bytes, int nreg, int slots)
{
    ResidentPlan p = {false, 0, 0, 0, 0};
    const int C4 = C / 4;
    if (C % 4 != 0 || C4 < 4 || C4 > 128 || (C4 & (C4 - 1)) != 0) return p;     // power of two, 16...512 channels
    const long long n4 = (long long)rows * C4;
    static const long long min_mb = [] { const char* v = getenv("HPF_BN_RES_MIN_MB"); return v ? atoll(v) : 16ll; }();
    if (n4 * 16 < (min_mb << 20)) return p;                                     // smaller tensors: the two-kernel path wins
    int sms = resident_sm_count();
    // one partial row per CTA must fit the caller's scratch (sized for the two-kernel path)
    const long long max_rows = scratch_bytes > 256 ? (long long)((scratch_bytes - 256) / ((size_t)8 * C4 * sizeof(float))) : 0;
    if (sms > max_rows) sms = (int)max_rows;
    if (sms < 64) return p;
    long long per = (n4 + sms - 1) / sms;
    per = (per + C4 - 1) / C4 * C4;
    const int iters = (int)((per + kResThreads - 1) / kResThreads);
    if (iters > nreg + kResSmemV / slots) return p;
    p.grid = (int)((n4 + per - 1) / per);
    p.iters = iters; p.per_cta = per;
    p.smem = iters > nreg ? (size_t)(iters - nreg) * slots * kResThreads * sizeof(float4) : 0;
    p.ok = true;
    return p;
}

void resident_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, const ResidentPlan& p, cudaStream_t st)
{
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3(p.grid); cfg->blockDim = dim3(kResThreads); cfg->dynamicSmemBytes = p.smem; cfg->stream = st;
    attr[0].id = cudaLaunchAttributeCooperative;     // all CTAs resident together: the barrier cannot wait for an unscheduled CTA
    attr[0].val.cooperative = 1;
    cfg->attrs = attr; cfg->numAttrs = 1;
}

}  // namespace

// BN+ReLU from an on-chip copy.  Both return cudaErrorNotSupported (nothing launched) when the tensor is smaller than
// 16 MB or does not fit the chip, the channel count is not a power of two in 16...512, or the device cannot launch
// cooperatively; the caller then takes the two-kernel path.  scratch as for bnrelu_fwd / bnrelu_bwd: the first 256
// bytes zero before the first use (the kernels leave word 0 zero; word 1 counts barrier generations; word 2 becomes 1
// if a barrier wait ever gave up, and the statistics / parameter gradients of that call are NaN).
cudaError_t bnrelu_fwd_resident(const float* x, const float* gamma, const float* beta, float eps, float* y, float* stats,
                                int64_t rows, int C, void* scratch, cudaStream_t st, int64_t* n_launch, bool relu)
{
    const ResidentPlan p = resident_plan(rows, C, bn_scratch_bytes(rows, C), kResRegV, 1);
    if (!p.ok) return cudaErrorNotSupported;
    unsigned int* sync = reinterpret_cast<unsigned int*>(scratch);
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + 256);
    const float floor = relu ? 0.f : -INFINITY;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[1];
    resident_config(&cfg, attr, p, st);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, bn_fwd_resident_kernel, reinterpret_cast<const float4*>(x), gamma, beta, eps,
                                             reinterpret_cast<float4*>(y), stats, (long long)rows * (C / 4), (long long)rows, C,
                                             p.per_cta, p.iters, sync, partials, floor);
    if (e == cudaSuccess && n_launch) *n_launch += 1;
    return e;
}

cudaError_t bnrelu_bwd_resident(const float* x, const float* dy, const float* gamma, const float* beta, const float* stats,
                                float* dx, const float* addend, bool accumulate, float* dgamma, float* dbeta, int64_t rows, int C,
                                void* scratch, cudaStream_t st, int64_t* n_launch, bool relu)
{
    // dz and xhat both on chip where they fit, else dz alone and a second read of x
    ResidentPlan p = resident_plan(rows, C, bn_scratch_bytes(rows, C), kResRegBwdBoth, 2);
    const bool both = p.ok;
    if (!both) p = resident_plan(rows, C, bn_scratch_bytes(rows, C), kResRegBwd, 1);
    if (!p.ok) return cudaErrorNotSupported;
    unsigned int* sync = reinterpret_cast<unsigned int*>(scratch);
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + 256);
    const float floor = relu ? 0.f : -INFINITY;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[1];
    resident_config(&cfg, attr, p, st);
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const float4* dy4 = reinterpret_cast<const float4*>(dy);
    const float4* ad4 = reinterpret_cast<const float4*>(addend);
    float4* dx4 = reinterpret_cast<float4*>(dx);
    const long long n4 = (long long)rows * (C / 4);
    const int acc = accumulate ? 1 : 0;
    cudaError_t e;
    if (both) e = cudaLaunchKernelEx(&cfg, bn_bwd_resident_kernel<true>, x4, dy4, gamma, beta, stats, ad4, dx4, acc, dgamma, dbeta, n4,
                                     (long long)rows, C, p.per_cta, p.iters, sync, partials, floor);
    else e = cudaLaunchKernelEx(&cfg, bn_bwd_resident_kernel<false>, x4, dy4, gamma, beta, stats, ad4, dx4, acc, dgamma, dbeta, n4,
                                (long long)rows, C, p.per_cta, p.iters, sync, partials, floor);
    if (e == cudaSuccess && n_launch) *n_launch += 1;
    return e;
}

}  // namespace hpf
