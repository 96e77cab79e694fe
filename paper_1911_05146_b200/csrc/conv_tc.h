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
    int direct;          // weight gradient: the kernel that feeds the TMA tiles to the tensor core as they land
    alignas(64) unsigned char storage[896];
};

// Batch-norm work folded into the forward kernel.
//   Output side: the kernel's output is the input of a BN.  Per tile and output channel the write-out forms the sum and
//   the sum of squares of what it stores (partials, [conv_tc_tiles(s, PASS_FWD)][2][channels] floats).
//     mode 1: the CTA that finishes last (ticket: one zeroed word, left zero) adds them in a fixed order and stores
//             mean[C], rstd[C] of the `rows` pixels to stats_out;
//     mode 3: the kernel leaves the partials only; the convolution that applies the BN adds them (in_mode 2).
//   Input side: the kernel's input tensor is the INPUT x of a BN+ReLU op whose output only this convolution reads.  The
//   kernel applies y = relu(gamma*(x-mean)*rstd+beta) to the activation tile on its way to the tensor core (the padding
//   ring stays zero) and stores y (in_y, needed by the backward pass) as a by-product: the BN+ReLU needs no kernel.
//     in_mode 1: in_stats holds mean / rstd (the producer ran mode 1);
//     in_mode 2: every CTA adds the producer's per-tile sums (in_partials, in_tiles rows, statistics over in_rows
//                pixels) in the same fixed order and the first CTA stores mean / rstd to in_stats.
struct ConvBnFuse {
    int mode = 0;
    float* partials = nullptr;
    unsigned int* ticket = nullptr;
    float* stats_out = nullptr;
    long long rows = 0;
    float eps = 0.f;
    int in_mode = 0;
    const float* in_gamma = nullptr;
    const float* in_beta = nullptr;
    float* in_stats = nullptr;
    float* in_y = nullptr;
    // weight gradient only: > 0 caps the CTAs of the launch (fewer pixel splits, each walking more tiles): less SM time
    // at a longer duration, for launches that run beside a chain of latency-bound kernels
    int wgrad_max_ctas = 0;
    // weight gradient only: 1 keeps the kernel that transposes its tiles in shared memory (a cross-check)
    int wgrad_transposing = 0;
    const float* in_partials = nullptr;
    int in_tiles = 0;
    long long in_rows = 0;
    float in_eps = 0.f;
    // forward / data gradient without BN work: room for splitting a long K loop over several CTAs (conv_tc_splitk_bytes;
    // the first kSplitKTicketBytes hold tickets, zero before the first use and left zero).  nullptr: never split.
    void* splitk = nullptr;
    size_t splitk_bytes = 0;
    // > 0: the launch will run inside a persistent cell kernel of this many CTAs (conv_tc_cell_launch): tiles per CTA are
    // chosen so that the launch is one round of that grid where tensor and shared memory allow
    // forward / data gradient: programmatic launch of the kernel's successor when the first accumulator is complete
    // instead of at the kernel's first instruction
    int pdl_late = 0;
    int cell_ctas = 0;
    unsigned int cell_smem = 0;          // dynamic shared memory such a CTA may use (0: what lets two of them share an SM)
};
constexpr size_t kSplitKTicketBytes = 4096;
// Bytes a forward (or data-gradient) launch of this shape wants for splitting its K loop; 0 when it would not split.
size_t conv_tc_splitk_bytes(const ConvShape& s, int pass, int passes);
// Whether the input-side fusion applies to this convolution.
bool conv_tc_can_fuse_bn_input(const ConvShape& s);
// Number of pixel tiles (= partial-sum rows) of the forward / data-gradient launch, and whether the fusion applies.
int conv_tc_tiles(const ConvShape& s, int pass);
bool conv_tc_can_fuse_bn(const ConvShape& s, int pass);

// passes = 3: error-compensated (hi*hi + lo*hi + hi*lo); passes = 1: single TF32 pass.
// pass = PASS_FWD:   out = conv(in, w) (+ extra); w_hi / w_lo = split weights [K][R][R][C]
// pass = PASS_DGRAD: out (+)= dgrad(in = dy) (+ extra); w_hi / w_lo = split rearranged weights [C][R][R][K]
// pass = PASS_WGRAD: out = wgrad(in = dy, in2 = x)
cudaError_t conv_tc_prepare(ConvTcPlan* plan, const ConvShape& s, int pass, int passes, const float* in, const float* in2,
                            const float* w_hi, const float* w_lo, float* out, const float* extra, bool accumulate, void* scratch,
                            const ConvBnFuse* fuse = nullptr);
cudaError_t conv_tc_launch(const ConvTcPlan* plan, DeviceStatus* status, cudaStream_t st, int64_t* n_launch);

// Persistent cell kernel: a list of prepared forward / data-gradient launches run one after the other by ONE resident grid
// with a grid-wide barrier between them (see conv_tc.cu).  conv_tc_cell_op writes the device-side record of a prepared
// launch (conv_tc_cell_op_bytes() bytes, to be copied to 64-byte aligned device memory) and reports what the launch needs;
// cudaErrorNotSupported: the launch exceeds what a cell CTA may hold.  The list is launched with the largest smem /
// tmem_cols of its records.  d_barrier: two zeroed words per stream of cells.
size_t conv_tc_cell_op_bytes();
cudaError_t conv_tc_cell_op(const ConvTcPlan* plan, DeviceStatus* status, void* dst_host, unsigned int* smem, unsigned int* tmem_cols,
                            unsigned int* ctas);
// Depth of the prepared forward / data-gradient launch's operand pipeline and the length of its K loop.
void conv_tc_plan_pipeline(const ConvTcPlan* plan, int* stages, int* k_iterations);
// CTAs of the cell kernel that can be resident on the current device at once with this much dynamic shared memory.
int conv_tc_cell_max_ctas(unsigned int smem);
cudaError_t conv_tc_cell_launch(const void* d_ops, int n_ops, int ctas, unsigned int smem, unsigned int tmem_cols, unsigned int* d_barrier,
                                DeviceStatus* status, cudaStream_t st, int64_t* n_launch);

// One convolution's weights inside the flat parameter vector.
struct WeightPrepEntry { long long w_off; int C, K, R, reserved; };
// For every table entry (device memory): w_hi/w_lo = hi/lo split of the weights, wt_hi/wt_lo = split of the weights
// rearranged for the data gradient (wt[c][R-1-r][R-1-s][k] = w[k][r][s][c]); all four use the entry's w_off.
cudaError_t conv_weight_prep(const float* params, float* w_hi, float* w_lo, float* wt_hi, float* wt_lo,
                             const WeightPrepEntry* d_table, int n_entries, int max_tiles, cudaStream_t st, int64_t* n_launch);
// 32 x 32 tiles the preparation kernel walks for one convolution (max_tiles above = the largest of the table)
int conv_weight_prep_tiles(int C, int K, int R);

cudaError_t conv_weight_prep_single(const float* w, float* w_hi, float* w_lo, float* wt_hi, float* wt_lo, int C, int K, int R,
                                    cudaStream_t st, int64_t* n_launch);

}  // namespace hpf
