// hpf_bnrelu_fwd_static: the fused BN(training)+ReLU forward for callers that cannot allocate.
//
// Every other entry point takes its scratch memory from the caller, who got it from cudaMalloc (or from
// a framework allocator sitting on it).  Some callers have no such option at the moment of the call: code
// running inside a region where allocation is forbidden or would synchronise the device (a real-time loop,
// a callback on a stream, a plug-in that was handed fixed input and output buffers and nothing else).
// For them the scratch of this one kernel lives in a fixed array inside the library's device image.
#include "../../include/hpf.h"
#include "hpf_kernels.h"

#include <atomic>
#include <cstdio>

namespace {

// Capacity of the built-in scratch.  It is part of the loaded module: every GPU that loads the library holds
// these bytes until the process exits, whether or not this entry point is ever called.
constexpr size_t kStaticScratchBytes = 2u << 20;

// In host code this name is only a handle for cudaGetSymbolAddress, not an address a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
// Device address of the array per device, looked up by the first call on that device.  Two host threads making that
// first call at the same moment both store the same value; the slot is atomic so that this is a defined program.
std::atomic<void*> g_scratch_addr[kMaxDevices];

}  // namespace

extern "C" int hpf_bnrelu_fwd_static(const float* d_x, const float* d_gamma, const float* d_beta, float eps, float* d_y,
                                      float* d_stats, int64_t rows, int32_t C, void* stream)
{
    using hpf::api_fail;
    using hpf::api_cuda_fail;
    if (!d_x || !d_gamma || !d_beta || !d_y || !d_stats) return api_fail(HPF_ERR_INVALID, "null argument");
    if (rows < 1 || C < 4 || C % 4) return api_fail(HPF_ERR_UNSUPPORTED, "channel count must be a multiple of 4");
    // sizes whose partial sums do not fit the built-in array are refused, never truncated
    if (hpf::bn_scratch_bytes(rows, C) > kStaticScratchBytes)
        return api_fail(HPF_ERR_WORKSPACE, "hpf_bnrelu_fwd_static: the partial sums of this size exceed the built-in scratch (hpf_static_scratch_bytes)");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return api_cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return api_fail(HPF_ERR_UNSUPPORTED, "device index beyond the table of this entry point");
    void* scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        // once per device, with that device current: the device address of the array in this device's module
        e = cudaGetSymbolAddress(&scratch, g_static_scratch);
        if (e != cudaSuccess) return api_cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if (!scratch) return api_fail(HPF_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_scratch_addr[dev].store(scratch, std::memory_order_release);
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the block ticket at its head must start at zero
    e = cudaMemsetAsync(scratch, 0, 256, st);
    if (e != cudaSuccess) return api_cuda_fail(e, "cudaMemsetAsync(static scratch head)");
    e = hpf::bnrelu_fwd(d_x, d_gamma, d_beta, eps, d_y, d_stats, rows, C, scratch, st, nullptr);
    if (e != cudaSuccess) return api_cuda_fail(e, "bnrelu_fwd on the static scratch");
    return HPF_OK;
}

extern "C" int hpf_static_scratch_bytes(size_t* bytes)
{
    if (!bytes) return hpf::api_fail(HPF_ERR_INVALID, "null argument");
    *bytes = kStaticScratchBytes;
    return HPF_OK;
}
