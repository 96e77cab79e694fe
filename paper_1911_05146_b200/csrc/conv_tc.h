// Tensor-core (tcgen05 / TMEM / TMA) convolution path, sm_100a.  See conv_tc.cu.
#pragma once
#include "hpf_kernels.h"

namespace hpf {

enum ConvPass { PASS_FWD = 0, PASS_DGRAD = 1, PASS_WGRAD = 2 };

// Whether the tensor-core kernels cover this shape for this pass.
bool conv_tc_supported(const ConvShape& s, int pass);

// Resolves the driver entry point used to encode tensor maps.  Needs a CUDA driver.
cudaError_t conv_tc_init();

size_t conv_tc_scratch_bytes(const ConvShape& s);

// A prepared launch: tensor maps are encoded once (they bake in the device pointers) and the kernel
// parameters are kept ready in `storage`.
struct ConvTcPlan {
    ConvShape s;
    int pass;
    int valid;
    alignas(64) unsigned char storage[640];
};

// pass = PASS_FWD:   out = conv(in, weights) (+ extra)
// pass = PASS_DGRAD: out (+)= dgrad(in = dy, weights = rearranged weights) (+ extra)
// pass = PASS_WGRAD: out = wgrad(in = dy, in2 = x)
cudaError_t conv_tc_prepare(ConvTcPlan* plan, const ConvShape& s, int pass, const float* in, const float* in2,
                            const float* weights, float* out, const float* extra, bool accumulate, void* scratch);
cudaError_t conv_tc_launch(const ConvTcPlan* plan, DeviceStatus* status, cudaStream_t st, int64_t* n_launch);

// wt[c][R-1-r][R-1-s][k] = w[k][r][s][c]  (the weights of the data gradient seen as a forward convolution)
cudaError_t conv_dgrad_weights(const float* w, float* wt, int C, int K, int R, cudaStream_t st, int64_t* n_launch);

}  // namespace hpf
