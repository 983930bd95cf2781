// onnx_conv2d_run_static: the convolution run call for callers that cannot hand the
// library a workspace because they cannot allocate device memory at that point: code
// running inside a real-time or safety-certified loop whose memory was fixed at start-up,
// a plugin hosted by a framework that owns the allocator, or a process whose device heap is
// already fully reserved.  Whatever scratch the descriptor's kernel needs lives in a fixed
// array inside the library image instead: the packed, TF32-rounded weights of the implicit-GEMM
// kernel, the TF32-rounded weights of the 1x1 GEMM kernel, or the gathered input copy of the
// gather-then-GEMM kernel.
#include <cuda_runtime.h>

#include <atomic>

#include "common.h"

using namespace onnxb;

namespace {

// 10 MiB: enough for the largest ResNet-50 layer (512 x 512 x 3 x 3 weights = 9 MiB packed).
// Every GPU on which the library is loaded carries this array until the process exits.
constexpr size_t kStaticScratchBytes = 10u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the array on the current device.  In host code the symbol name is only a
// handle, not a device pointer, so the address must be asked for, once per device.
void *static_scratch_ptr() {
    static std::atomic<void *> ptrs[64];      // per device; every thread that races here stores the same value
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    void *cached = ptrs[dev].load(std::memory_order_acquire);
    if (!cached) {
        if (cudaGetSymbolAddress(&cached, g_static_scratch) != cudaSuccess) return nullptr;
        ptrs[dev].store(cached, std::memory_order_release);
    }
    return cached;
}

}  // namespace

extern "C" size_t onnx_conv2d_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" onnxb_status onnx_conv2d_run_static(onnxb_conv2d_desc_t d, const float *X, const float *W,
                                               const float *B, float *Y, void *cuda_stream) {
    if (!d) return ONNXB_ERR_NULL;
    if (d->workspace_bytes == 0)   // this descriptor's kernel needs no scratch at all
        return onnx_conv2d_run(d, X, W, B, Y, nullptr, 0, cuda_stream);
    if (d->workspace_bytes > kStaticScratchBytes) return ONNXB_ERR_WORKSPACE;
    void *scratch = static_scratch_ptr();
    if (!scratch) return ONNXB_ERR_CUDA;
    // Each family's first kernel (weight packing, weight rounding or the input gather) rewrites
    // every byte of the scratch that its second kernel reads (zero padding included), so nothing
    // left behind by an earlier call can leak into this one.
    return onnx_conv2d_run(d, X, W, B, Y, scratch, kStaticScratchBytes, cuda_stream);
}
