// onnxb_probe_tf32_mma_rate: a measurement aid, not part of the operators.  It times the
// tensor pipe alone: one thread per CTA issues tcgen05.mma kind::tf32 instructions of shape
// 128 x N x 8 back to back on operands that already sit in shared memory (zeros; no loads, no
// epilogue), on every SM at once, and reports SM cycles per instruction.  That is the ceiling
// any kernel of this library built from the same instruction can reach for that N, and the
// denominator the roofline figures for the TF32 path are compared with.
#include <cuda_runtime.h>

#include "common.h"
#include "tc_common.cuh"
#include "tc_host.h"

namespace onnxb {
namespace {

using namespace tc;

constexpr int kProbeOperandBytes = 64 * 1024;      // each of A and B
constexpr int kProbeSmem = 2048 + 2 * kProbeOperandBytes;

// K-major operands without swizzle, rows 16 bytes apart (the convolution kernel's layout); sixteen
// different start addresses per round, as the filter taps of a convolution give.
__global__ void __launch_bounds__(128, 1)
tf32_mma_rate_kernel(int n, int rounds, long long *cycles, unsigned int *err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t *bar = reinterpret_cast<uint64_t *>(smem);
    uint32_t *holder = reinterpret_cast<uint32_t *>(smem + 64);
    uint8_t *A = smem + 1024, *B = A + kProbeOperandBytes;
    for (int i = threadIdx.x; i < 2 * kProbeOperandBytes / 4; i += blockDim.x) reinterpret_cast<float *>(A)[i] = 0.f;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_fence_init();
    }
    if (threadIdx.x < 32) {
        tmem_alloc(holder, 512);
        tmem_relinquish();
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = *holder;
    if (threadIdx.x == 0) {
        const uint32_t idesc = make_idesc_tf32(128, n, 0, 0);
        const long long t0 = clock64();
        for (int it = 0; it < rounds; ++it) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                // A: 128 rows from a shifted start (chunks 16 KB apart); B: n rows, chunks n*16 bytes apart
                const uint64_t ad = make_smem_desc(smem_u32(A) + (uint32_t)j * 496u, 16384, 128, kSwizzleNone);
                const uint64_t bd = make_smem_desc(smem_u32(B) + (uint32_t)(j & 3) * (uint32_t)n * 32u, (uint32_t)n * 16u,
                                                   128, kSwizzleNone);
                mma_tf32(tm + (uint32_t)((j & 1) * 256), ad, bd, idesc, 1);
            }
        }
        mma_commit(bar);
        mbar_wait(bar, 0, err, 30);
        cycles[blockIdx.x] = clock64() - t0;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) {
        tc_fence_after_sync();
        tmem_dealloc(tm, 512);
    }
}

// One CTA waits on an mbarrier that nothing ever arrives on, with a short limit.  The wait gives up,
// records code 31 in the error word and the kernel returns normally: the bounded-wait error path of the
// tensor-core kernels, exercised without a fault, a trap or an endless loop.
__global__ void wait_timeout_kernel(long long limit_cycles, unsigned int *err) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(&bar, 0, err, 31, limit_cycles);
    __syncthreads();
}

}  // namespace
}  // namespace onnxb

extern "C" onnxb_status onnxb_probe_wait_timeout(long long limit_cycles, void *cuda_stream) {
    using namespace onnxb;
    if (limit_cycles < 1 || limit_cycles > 100000000LL) return ONNXB_ERR_ATTR;     // at most ~50 ms
    unsigned int *err = device_status_ptr();
    if (!err) return ONNXB_ERR_CUDA;
    wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(limit_cycles, err);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? ONNXB_OK : ONNXB_ERR_CUDA;
}

extern "C" onnxb_status onnxb_probe_tf32_mma_rate(int n, int instructions, double *cycles_per_instruction,
                                                  void *cuda_stream) {
    using namespace onnxb;
    if (!cycles_per_instruction) return ONNXB_ERR_NULL;
    if (n < 16 || n > 256 || n % 16 || instructions < 16 || instructions > (1 << 20)) return ONNXB_ERR_ATTR;
    unsigned int *err = device_status_ptr();
    if (!err) return ONNXB_ERR_CUDA;
    const int sms = tc_host::num_sms();
    long long *dev = nullptr;
    // a measurement call, not a run call: it allocates its small result buffer and synchronises
    if (cudaMalloc(&dev, sizeof(long long) * sms) != cudaSuccess) return ONNXB_ERR_CUDA;
    onnxb_status st = ONNXB_OK;
    const int rounds = (instructions + 15) / 16;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaFuncSetAttribute(tf32_mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem) != cudaSuccess)
        st = ONNXB_ERR_CUDA;
    for (int rep = 0; rep < 2 && st == ONNXB_OK; ++rep) {      // the second launch is the measured one
        tf32_mma_rate_kernel<<<sms, 128, kProbeSmem, s>>>(n, rounds, dev, err);
        count_launch();
        if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) st = ONNXB_ERR_CUDA;
    }
    if (st == ONNXB_OK) {
        long long host[1024];
        const int cnt = sms < 1024 ? sms : 1024;
        if (cudaMemcpy(host, dev, sizeof(long long) * cnt, cudaMemcpyDeviceToHost) != cudaSuccess) {
            st = ONNXB_ERR_CUDA;
        } else {
            long long worst = 0;
            for (int i = 0; i < cnt; ++i) worst = host[i] > worst ? host[i] : worst;
            *cycles_per_instruction = (double)worst / ((double)rounds * 16.0);
        }
    }
    cudaFree(dev);
    return st;
}
