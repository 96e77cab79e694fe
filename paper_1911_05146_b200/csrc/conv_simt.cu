// CUDA-core (fp32 FMA) convolution kernels: forward, data gradient, weight gradient for any
// kernel size / stride / padding / channel count.  They serve the 3-channel stem convolution
// (whose reduction length 27 or 147 cannot feed the tensor-core path: a 12-byte pixel is no legal
// TMA row), channel counts that are not multiples of 16, and as an fp32 cross-check of the
// tensor-core kernels.  One kernel, three addressing modes of the same 64x64x16 tiled GEMM.
#include "hpf_kernels.h"

namespace hpf {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, THREADS = 256;

enum { MODE_FWD = 0, MODE_DGRAD = 1, MODE_WGRAD = 2 };

struct SimtArgs {
    const float* a;        // fwd: x      dgrad: dy     wgrad: dy
    const float* b;        // fwd: w      dgrad: w      wgrad: x
    float* out;            // fwd: y      dgrad: dx     wgrad: partials [splits][K][R*R*C]
    const float* extra;    // fwd: residual, dgrad: addend (nullable)
    int accumulate;        // dgrad: dx += result
    ConvShape s;
    int Md, Nd, Kd;        // GEMM extents
    int k_per_split;       // wgrad: pixels per grid.z slice
};

// A(m, kk) of the GEMM view
template <int MODE>
__device__ __forceinline__ float load_a(const SimtArgs& g, int m, int kk)
{
    const ConvShape& s = g.s;
    if (MODE == MODE_FWD) {            // m = (n,p,q), kk = (r,s,c)
        const int c = kk % s.C; int t = kk / s.C;
        const int ss = t % s.R, rr = t / s.R;
        const int q = m % s.Q; t = m / s.Q;
        const int p = t % s.P, n = t / s.P;
        const int ih = p * s.stride + rr - s.pad, iw = q * s.stride + ss - s.pad;
        if (ih < 0 || ih >= s.H || iw < 0 || iw >= s.W) return 0.f;
        return __ldg(&g.a[(((int64_t)n * s.H + ih) * s.W + iw) * s.C + c]);
    } else if (MODE == MODE_DGRAD) {   // m = (n,h,w), kk = (r,s,k)
        const int k = kk % s.K; int t = kk / s.K;
        const int ss = t % s.R, rr = t / s.R;
        const int w = m % s.W; t = m / s.W;
        const int h = t % s.H, n = t / s.H;
        const int tp = h + s.pad - rr, tq = w + s.pad - ss;
        if (tp < 0 || tq < 0 || tp % s.stride || tq % s.stride) return 0.f;
        const int p = tp / s.stride, q = tq / s.stride;
        if (p >= s.P || q >= s.Q) return 0.f;
        return __ldg(&g.a[(((int64_t)n * s.P + p) * s.Q + q) * s.K + k]);
    } else {                           // m = k (output channel), kk = pixel (n,p,q)
        return __ldg(&g.a[(int64_t)kk * s.K + m]);
    }
}

// B(kk, n) of the GEMM view
template <int MODE>
__device__ __forceinline__ float load_b(const SimtArgs& g, int kk, int n)
{
    const ConvShape& s = g.s;
    if (MODE == MODE_FWD) {            // w[n][kk]
        return __ldg(&g.b[(int64_t)n * g.Kd + kk]);
    } else if (MODE == MODE_DGRAD) {   // kk = (r,s,k), n = c: w[k][r][s][c]
        const int k = kk % s.K; const int t = kk / s.K;
        return __ldg(&g.b[((int64_t)k * s.R * s.R + t) * s.C + n]);
    } else {                           // kk = pixel (n,p,q), n = (r,s,c): x[n, p*st+r-pad, q*st+s-pad, c]
        const int c = n % s.C; int t = n / s.C;
        const int ss = t % s.R, rr = t / s.R;
        const int q = kk % s.Q; t = kk / s.Q;
        const int p = t % s.P, img = t / s.P;
        const int ih = p * s.stride + rr - s.pad, iw = q * s.stride + ss - s.pad;
        if (ih < 0 || ih >= s.H || iw < 0 || iw >= s.W) return 0.f;
        return __ldg(&g.b[(((int64_t)img * s.H + ih) * s.W + iw) * s.C + c]);
    }
}

template <int MODE>
__global__ void __launch_bounds__(THREADS) conv_simt_kernel(SimtArgs g)
{
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    int k_begin = 0, k_end = g.Kd;
    if (MODE == MODE_WGRAD) {
        k_begin = blockIdx.z * g.k_per_split;
        k_end = k_begin + g.k_per_split;
        if (k_end > g.Kd) k_end = g.Kd;
    }
    const int ty = tid / 16, tx = tid % 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = k_begin; k0 < k_end; k0 += BK) {
        // 64x16 elements of A and of B, 4 each per thread
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = tid + e * THREADS;
            int kk, mm;
            if (MODE == MODE_WGRAD) { mm = idx % BM; kk = idx / BM; }   // A contiguous along m (channels of dy)
            else { kk = idx % BK; mm = idx / BK; }                      // A contiguous along kk (channels)
            const int m = m0 + mm, k = k0 + kk;
            As[kk][mm] = (m < g.Md && k < k_end) ? load_a<MODE>(g, m, k) : 0.f;
            int kb, nn;
            if (MODE == MODE_FWD) { kb = idx % BK; nn = idx / BK; }     // w[n][kk]: contiguous along kk
            else { nn = idx % BN; kb = idx / BN; }                      // contiguous along n
            const int n = n0 + nn, k2 = k0 + kb;
            Bs[kb][nn] = (n < g.Nd && k2 < k_end) ? load_b<MODE>(g, k2, n) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= g.Md) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= g.Nd) continue;
            float v = acc[i][j];
            if (MODE == MODE_WGRAD) {
                g.out[((int64_t)blockIdx.z * g.Md + m) * g.Nd + n] = v;
            } else {
                const int64_t o = (int64_t)m * g.Nd + n;
                if (g.extra) v += __ldg(&g.extra[o]);
                if (MODE == MODE_DGRAD && g.accumulate) v += g.out[o];
                g.out[o] = v;
            }
        }
    }
}

// dw[i] = sum over splits (ascending) of partials[z][i]
__global__ void __launch_bounds__(THREADS)
wgrad_reduce_kernel(const float* __restrict__ partials, float* __restrict__ dw, int64_t n, int splits)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float s = 0.f;
#pragma unroll 8
        for (int z = 0; z < splits; ++z) s += __ldcg(&partials[(int64_t)z * n + i]);
        dw[i] = s;
    }
}

struct WgradSplit { int splits, k_per_split; };
WgradSplit wgrad_split(const ConvShape& s)
{
    const int64_t pixels = (int64_t)s.N * s.P * s.Q;
    const int64_t outs = (int64_t)s.K * s.R * s.R * s.C;
    int64_t splits = pixels / 1024;                       // >= 1024 pixels per slice
    // few output tiles (a stem convolution: one to three): the slices are what fills the GPU, down to 128 pixels each
    const int64_t out_tiles = (int64_t)((s.K + BM - 1) / BM) * ((s.R * s.R * s.C + BN - 1) / BN);
    if (splits * out_tiles < 296) splits = (296 + out_tiles - 1) / out_tiles;
    if (splits > pixels / 128) splits = pixels / 128;
    const int64_t cap = (int64_t)(32 << 20) / (outs * 4) ;  // partials <= 32 MiB
    if (splits > cap) splits = cap;
    if (splits > 256) splits = 256;
    if (splits < 1) splits = 1;
    int64_t kps = (pixels + splits - 1) / splits;
    kps = (kps + BK - 1) / BK * BK;
    WgradSplit r;
    r.k_per_split = (int)kps;
    r.splits = (int)((pixels + kps - 1) / kps);
    return r;
}

inline void count(int64_t* n_launch, int k) { if (n_launch) *n_launch += k; }

}  // namespace

size_t conv_simt_scratch_bytes(const ConvShape& s)
{
    const WgradSplit w = wgrad_split(s);
    return (size_t)w.splits * s.K * s.R * s.R * s.C * sizeof(float);
}

cudaError_t conv_fwd_simt(const float* x, const float* w, float* y, const float* residual, const ConvShape& s,
                          cudaStream_t st, int64_t* n_launch)
{
    SimtArgs g{x, w, y, residual, 0, s, s.N * s.P * s.Q, s.K, s.R * s.R * s.C, 0};
    dim3 grid((g.Md + BM - 1) / BM, (g.Nd + BN - 1) / BN, 1);
    conv_simt_kernel<MODE_FWD><<<grid, THREADS, 0, st>>>(g);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t conv_dgrad_simt(const float* dy, const float* w, float* dx, const float* addend, bool accumulate,
                            const ConvShape& s, cudaStream_t st, int64_t* n_launch)
{
    SimtArgs g{dy, w, dx, addend, accumulate ? 1 : 0, s, s.N * s.H * s.W, s.C, s.R * s.R * s.K, 0};
    dim3 grid((g.Md + BM - 1) / BM, (g.Nd + BN - 1) / BN, 1);
    conv_simt_kernel<MODE_DGRAD><<<grid, THREADS, 0, st>>>(g);
    count(n_launch, 1);
    return cudaGetLastError();
}

cudaError_t conv_wgrad_simt(const float* x, const float* dy, float* dw, const ConvShape& s, void* scratch,
                            cudaStream_t st, int64_t* n_launch)
{
    const WgradSplit ws = wgrad_split(s);
    SimtArgs g{dy, x, reinterpret_cast<float*>(scratch), nullptr, 0, s, s.K, s.R * s.R * s.C, s.N * s.P * s.Q,
               ws.k_per_split};
    dim3 grid((g.Md + BM - 1) / BM, (g.Nd + BN - 1) / BN, ws.splits);
    conv_simt_kernel<MODE_WGRAD><<<grid, THREADS, 0, st>>>(g);
    const int64_t n = (int64_t)s.K * s.R * s.R * s.C;
    int nb = (int)((n + THREADS - 1) / THREADS);
    if (nb > 1184) nb = 1184;
    wgrad_reduce_kernel<<<nb, THREADS, 0, st>>>(reinterpret_cast<const float*>(scratch), dw, n, ws.splits);
    count(n_launch, 2);
    return cudaGetLastError();
}

}  // namespace hpf
