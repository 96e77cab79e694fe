// hpf_bnrelu_fwd_static: the fused BN(training)+ReLU forward for callers that cannot allocate.
//
// Every other entry point takes its scratch memory from the caller, who got it from cudaMalloc (or from
// a framework allocator sitting on it).  Some callers have no such option at the moment of the call: code
// running inside a region where allocation is forbidden or would synchronise the device (a real-time loop,
// a callback on a stream, a plug-in that was handed fixed input and output buffers and nothing else).
// For them the scratch of this one kernel lives in a fixed array inside the library's device image.
#include "../../include/hpf.h"
#include "hpf_kernels.h"

#include <cstdio>
#include <string>

namespace {

// Capacity of the built-in scratch.  It is part of the loaded module: every GPU that loads the library holds
// these bytes until the process exits, whether or not this entry point is ever called.
constexpr size_t kStaticScratchBytes = 2u << 20;

// In host code this name is only a handle for cudaGetSymbolAddress, not an address a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};

}  // namespace

extern "C" int hpf_bnrelu_fwd_static(const float* d_x, const float* d_gamma, const float* d_beta, float eps, float* d_y,
                                      float* d_stats, int64_t rows, int32_t C, void* stream)
{
    if (!d_x || !d_gamma || !d_beta || !d_y || !d_stats) return HPF_ERR_INVALID;
    if (rows < 1 || C < 4 || C % 4) return HPF_ERR_UNSUPPORTED;
    // sizes whose partial sums do not fit the built-in array are refused, never truncated
    if (hpf::bn_scratch_bytes(rows, C) > kStaticScratchBytes) return HPF_ERR_WORKSPACE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HPF_ERR_CUDA;
    if (!g_scratch_addr[dev]) {
        // once per device, with that device current: the device address of the array in this device's module
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return HPF_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    void* scratch = g_scratch_addr[dev];
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the block ticket at its head must start at zero
    if (cudaMemsetAsync(scratch, 0, 256, st) != cudaSuccess) return HPF_ERR_CUDA;
    if (hpf::bnrelu_fwd(d_x, d_gamma, d_beta, eps, d_y, d_stats, rows, C, scratch, st, nullptr) != cudaSuccess) return HPF_ERR_CUDA;
    return HPF_OK;
}

extern "C" int hpf_static_scratch_bytes(size_t* bytes)
{
    if (!bytes) return HPF_ERR_INVALID;
    *bytes = kStaticScratchBytes;
    return HPF_OK;
}
