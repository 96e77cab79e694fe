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

// A prepared launch: tensor maps are encoded once (they bake in the device pointers).
struct ConvTcPlan {
    alignas(64) unsigned char tmap_a[128];   // activation operand (x or dy)
    alignas(64) unsigned char tmap_b[128];   // weight operand (fwd/dgrad) or second activation operand (wgrad)
    ConvShape s;
    int pass;
    int valid;
    // tile geometry (see conv_tc.cu)
    int box_w, box_h, box_n;      // pixel box of one M tile
    int tiles_w, tiles_h, tiles_n;
    int kchunk;                   // channels per K step (16 or 32)
    int n_kchunks;                // c_in / kchunk
    int swizzle_bytes;            // 64 or 128
    int stages;
    int splits;                   // wgrad: pixel-tile slices (grid.y)
    unsigned int smem_bytes;
    unsigned int tmem_cols;
    const float* in;              // fwd: x, dgrad: dy, wgrad: dy
    const float* in2;             // wgrad: x
    const float* weights;         // fwd: w, dgrad: transformed weights
    float* out;                   // fwd: y, dgrad: dx, wgrad: dw
    const float* extra;           // fwd: residual, dgrad: addend (nullable)
    int accumulate;
    void* scratch;                // wgrad partials
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
