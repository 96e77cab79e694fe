// Tensor-core convolution path (placeholder until the tcgen05 kernels land): reports every shape as
// outside its reach, so all convolutions run on the CUDA-core kernels.
#include "conv_tc.h"

namespace hpf {

bool conv_tc_supported(const ConvShape&, int) { return false; }
cudaError_t conv_tc_init() { return cudaSuccess; }
size_t conv_tc_scratch_bytes(const ConvShape&) { return 0; }
cudaError_t conv_tc_prepare(ConvTcPlan* plan, const ConvShape&, int, const float*, const float*, const float*, float*,
                            const float*, bool, void*)
{
    plan->valid = 0;
    return cudaErrorNotSupported;
}
cudaError_t conv_tc_launch(const ConvTcPlan*, DeviceStatus*, cudaStream_t, int64_t*) { return cudaErrorNotSupported; }

namespace {
__global__ void dgrad_weights_kernel(const float* __restrict__ w, float* __restrict__ wt, int C, int K, int R)
{
    const int64_t total = (int64_t)K * R * R * C;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += stride) {
        // o indexes wt[c][r'][s'][k]
        const int k = (int)(o % K);
        int64_t t = o / K;
        const int s2 = (int)(t % R); t /= R;
        const int r2 = (int)(t % R);
        const int c = (int)(t / R);
        wt[o] = __ldg(&w[(((int64_t)k * R + (R - 1 - r2)) * R + (R - 1 - s2)) * C + c]);
    }
}
}  // namespace

cudaError_t conv_dgrad_weights(const float* w, float* wt, int C, int K, int R, cudaStream_t st, int64_t* n_launch)
{
    const int64_t total = (int64_t)K * R * R * C;
    int nb = (int)((total + 255) / 256);
    if (nb > 592) nb = 592;
    dgrad_weights_kernel<<<nb, 256, 0, st>>>(w, wt, C, K, R);
    if (n_launch) *n_launch += 1;
    return cudaGetLastError();
}

}  // namespace hpf
