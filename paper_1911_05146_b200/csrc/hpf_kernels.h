// Internal launcher interface between the host scheduler and the CUDA kernels.
// Every launcher only enqueues on `st`, returns the launch status and adds the
// number of kernels it launched to *n_launch (if non-null).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

namespace hpf {

struct ConvShape {
    int N, H, W, C;      // input  [N][H][W][C]
    int K, R, stride, pad;
    int P, Q;            // output [N][P][Q][K]
};
inline ConvShape make_conv_shape(int N, int H, int W, int C, int K, int R, int stride, int pad)
{
    ConvShape s{N, H, W, C, K, R, stride, pad, (H + 2 * pad - R) / stride + 1, (W + 2 * pad - R) / stride + 1};
    return s;
}

// Programmatic dependent launch.  The step is a long chain of small dependent kernels, so the gap between the end
// of one and the start of the next is a sizeable part of the critical path.  Hot kernels are launched with the
// programmatic-serialisation attribute: such a kernel may be scheduled while its predecessor in the stream is
// still running, executes its prologue (barrier and tensor-memory set-up, parameter and descriptor fetches), and
// blocks in pdl_wait() until the predecessor has completed and its writes are visible.  Every kernel launched
// this way calls pdl_wait() before its first read or write of global data.
// Per host thread: the model whose phase is being enqueued sets it for the duration of the enqueue (PdlScope).
extern thread_local bool g_pdl_enabled;
struct PdlScope {
    bool saved;
    explicit PdlScope(bool on) : saved(g_pdl_enabled) { g_pdl_enabled = on; }
    ~PdlScope() { g_pdl_enabled = saved; }
    PdlScope(const PdlScope&) = delete;
    PdlScope& operator=(const PdlScope&) = delete;
};
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = g_pdl_enabled ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Failure bookkeeping of the C ABI (hpf_model.cu): records the text hpf_last_error() returns on the calling thread
// and hands the status back, so that every entry point, whichever file it lives in, reports through one place.
int api_fail(int status, const char* what);
int api_cuda_fail(cudaError_t e, const char* where);

// Device-side status word shared by all kernels that have bounded waits.
// 0 = fine; anything else = where a wait gave up (see conv_tc.cu).
struct DeviceStatus { unsigned int code; unsigned int detail; };

// ---------------- memory-bound kernels (kernels_mem.cu) ----------------
size_t bn_scratch_bytes(int64_t rows, int C);
// scratch: first 256 bytes hold the block ticket (must be zero before the first use; the kernels
// leave it zero), the rest holds per-block partial sums.
// relu = false: batch normalisation without the activation (the post-activation block's second BN)
cudaError_t bnrelu_fwd(const float* x, const float* gamma, const float* beta, float eps, float* y, float* stats,
                       int64_t rows, int C, void* scratch, cudaStream_t st, int64_t* n_launch, bool relu = true);
cudaError_t bnrelu_bwd(const float* x, const float* dy, const float* gamma, const float* beta, const float* stats,
                       float* dx, const float* addend, bool accumulate, float* dgamma, float* dbeta,
                       int64_t rows, int C, void* scratch, cudaStream_t st, int64_t* n_launch, bool relu = true,
                       bool x_is_old = false);
// x_is_old: x, stats, gamma and beta were complete before the kernels just ahead of this call in the stream were
// enqueued (forward results read by a backward pass), so the kernel may fetch them while its predecessor still runs.
// The forward from an on-chip copy of the tensor (bn_resident.cu): one cooperative launch that holds every SM, for
// single-op calls on tensors of 8 MB and more that fit the chip.  cudaErrorNotSupported = not applicable, nothing
// launched.  Same scratch convention; words 1 and 2 of the scratch are used besides the ticket.
cudaError_t bnrelu_fwd_resident(const float* x, const float* gamma, const float* beta, float eps, float* y, float* stats,
                                int64_t rows, int C, void* scratch, cudaStream_t st, int64_t* n_launch, bool relu = true);
cudaError_t bnrelu_bwd_resident(const float* x, const float* dy, const float* gamma, const float* beta, const float* stats,
                                float* dx, const float* addend, bool accumulate, float* dgamma, float* dbeta, int64_t rows, int C,
                                void* scratch, cudaStream_t st, int64_t* n_launch, bool relu = true);
extern thread_local bool g_bn_cluster;   // single-launch cluster kernel for micro-batch sized BN backward (default on)
struct BnClusterScope {
    bool saved;
    explicit BnClusterScope(bool on) : saved(g_bn_cluster) { g_bn_cluster = on; }
    ~BnClusterScope() { g_bn_cluster = saved; }
    BnClusterScope(const BnClusterScope&) = delete;
    BnClusterScope& operator=(const BnClusterScope&) = delete;
};
// stand-alone ReLU: y = max(x, 0); dx (+= if accumulate) = dy * [x > 0] (+ addend)
cudaError_t relu_fwd(const float* x, float* y, int64_t n, cudaStream_t st, int64_t* n_launch);
cudaError_t relu_bwd(const float* x, const float* dy, float* dx, const float* addend, bool accumulate, int64_t n, cudaStream_t st,
                     int64_t* n_launch);
// The forward's second half alone: the statistics (mean[C], rstd[C]) were left by the convolution kernel that produced x.
cudaError_t bnrelu_fwd_apply(const float* x, const float* gamma, const float* beta, const float* stats, float* y,
                             int64_t rows, int C, cudaStream_t st, int64_t* n_launch);
cudaError_t add_fwd(const float* a, const float* b, float* out, int64_t n, cudaStream_t st, int64_t* n_launch);
// dst (+)= src
cudaError_t grad_accumulate(float* dst, const float* src, int64_t n, bool accumulate, cudaStream_t st, int64_t* n_launch);
cudaError_t grad_average(const float* slots, float* out, int M, int64_t G, cudaStream_t st, int64_t* n_launch);
// gbar = average of the M slots (stored to gavg unless null); v <- mu*v - lr*(gbar + wd*theta); theta <- theta + v
cudaError_t sgd_momentum(const float* slots, float* gavg, float* theta, float* vel, int M, int64_t G, float lr, float mu,
                         float wd, cudaStream_t st, int64_t* n_launch);
// writes the device's nanosecond timer to *slot (one thread)
cudaError_t stamp_time(unsigned long long* slot, cudaStream_t st, int64_t* n_launch);
cudaError_t loss_average(const float* loss_slots, float* out, int M, cudaStream_t st, int64_t* n_launch);
cudaError_t maxpool_fwd(const float* x, float* y, ConvShape s, cudaStream_t st, int64_t* n_launch);
cudaError_t maxpool_bwd(const float* x, const float* dy, float* dx, bool accumulate, ConvShape s, cudaStream_t st,
                        int64_t* n_launch);
// head: a [b][HW][C]; pooled scratch [b][C]; persample scratch [b]
cudaError_t head_fwd(const float* a, const float* Wfc, const float* bias, const int32_t* labels, float* logits,
                     float* pooled, float* persample, float* loss_slot, int b, int HW, int C, int ncls,
                     cudaStream_t st, int64_t* n_launch);
cudaError_t head_bwd(const float* Wfc, const int32_t* labels, const float* logits, const float* pooled,
                     float* dlogits, float* da, float* dW, float* dbias, int b, int HW, int C, int ncls,
                     cudaStream_t st, int64_t* n_launch);

// ---------------- CUDA-core convolutions (conv_simt.cu) ----------------
size_t conv_simt_scratch_bytes(const ConvShape& s);
// y = conv(x, w) (+ residual)
cudaError_t conv_fwd_simt(const float* x, const float* w, float* y, const float* residual, const ConvShape& s,
                          cudaStream_t st, int64_t* n_launch);
// dx (+= if accumulate) = dgrad(dy, w) (+ addend)
cudaError_t conv_dgrad_simt(const float* dy, const float* w, float* dx, const float* addend, bool accumulate,
                            const ConvShape& s, cudaStream_t st, int64_t* n_launch);
cudaError_t conv_wgrad_simt(const float* x, const float* dy, float* dw, const ConvShape& s, void* scratch,
                            cudaStream_t st, int64_t* n_launch);

}  // namespace hpf
