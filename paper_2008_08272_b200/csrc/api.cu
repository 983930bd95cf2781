// C-ABI run calls: argument checks, dispatch, launch.  Nothing here allocates
// device memory or synchronises (except onnxb_last_device_status, by contract).
#include <cuda_runtime.h>

#include "common.h"

using namespace onnxb;

namespace onnxb {
// Error word set by bounded device-side waits that ran out.
__device__ unsigned int g_device_status_word = 0;
}  // namespace onnxb

static inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

extern "C" onnxb_status onnx_conv2d_run(onnxb_conv2d_desc_t d, const float *X, const float *W,
                                        const float *B, float *Y, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream) {
    if (!d || !X || !W || !Y) return ONNXB_ERR_NULL;
    if ((d->g.has_bias != 0) != (B != nullptr)) return ONNXB_ERR_NULL;
    if (d->workspace_bytes > 0 && (!workspace || workspace_bytes < d->workspace_bytes)) return ONNXB_ERR_WORKSPACE;
    if (misaligned(X) || misaligned(W) || misaligned(B) || misaligned(Y) || misaligned(workspace))
        return ONNXB_ERR_UNSUPPORTED;

    int err;
    switch (d->family) {
        case ONNXB_KERNEL_SIMT_DEPTHWISE:
            err = launch_simt_depthwise(d->g, X, W, B, Y, cuda_stream);
            break;
        case ONNXB_KERNEL_SIMT_DIRECT:
            err = launch_simt_conv(d->g, X, W, B, Y, cuda_stream);
            break;
        default:
            return ONNXB_ERR_UNSUPPORTED;
    }
    return err == 0 ? ONNXB_OK : ONNXB_ERR_CUDA;
}

extern "C" size_t onnx_gemm_workspace_bytes(int, int, int64_t, int64_t, int64_t) { return 0; }

extern "C" onnxb_status onnx_gemm_run(int transA, int transB, float alpha, float beta, int64_t M, int64_t N,
                                      int64_t K, const float *A, const float *B, const float *C, int c_rank,
                                      const int64_t *c_dims, int fuse_relu, float *Y, void *workspace,
                                      size_t workspace_bytes, void *cuda_stream) {
    (void)workspace_bytes;
    if (!A || !B || !Y) return ONNXB_ERR_NULL;
    if (M < 1 || N < 1 || K < 1) return ONNXB_ERR_SHAPE;
    const int64_t lim = 2147483647LL;
    if (M > lim || N > lim || K > lim || M * K > lim || K * N > lim || M * N > lim) return ONNXB_ERR_UNSUPPORTED;

    GemmProblem p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.transA = transA != 0; p.transB = transB != 0;
    p.alpha = alpha; p.beta = beta; p.relu = fuse_relu != 0;
    p.c_stride_i = p.c_stride_j = 0;
    if (C) {
        if (c_rank < 0 || c_rank > 2 || (c_rank > 0 && !c_dims)) return c_rank > 0 && !c_dims ? ONNXB_ERR_NULL : ONNXB_ERR_SHAPE;
        // numpy-style one-directional broadcast: align C's dims with the trailing axes of [M,N]
        int64_t rows = 1, cols = 1;
        if (c_rank == 1) cols = c_dims[0];
        if (c_rank == 2) { rows = c_dims[0]; cols = c_dims[1]; }
        if ((rows != 1 && rows != M) || (cols != 1 && cols != N)) return ONNXB_ERR_SHAPE;
        p.c_stride_i = rows == 1 ? 0 : cols;
        p.c_stride_j = cols == 1 ? 0 : 1;
    }
    if (misaligned(A) || misaligned(B) || misaligned(C) || misaligned(Y) || misaligned(workspace))
        return ONNXB_ERR_UNSUPPORTED;

    const int err = launch_simt_gemm(p, A, B, C, Y, cuda_stream);
    return err == 0 ? ONNXB_OK : ONNXB_ERR_CUDA;
}

extern "C" onnxb_status onnxb_last_device_status(void *cuda_stream) {
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return ONNXB_ERR_CUDA;
    unsigned int word = 0;
    if (cudaMemcpyFromSymbol(&word, g_device_status_word, sizeof word) != cudaSuccess) return ONNXB_ERR_CUDA;
    if (word != 0) {
        const unsigned int zero = 0;
        cudaMemcpyToSymbol(g_device_status_word, &zero, sizeof zero);
        return ONNXB_ERR_DEVICE_TIMEOUT;
    }
    return ONNXB_OK;
}
