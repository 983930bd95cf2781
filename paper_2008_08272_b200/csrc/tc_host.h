// Host-side interface of the tensor-core family.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "common.h"

namespace onnxb {

// D[b] (M x N) = A'[b] (M x K) * B'[b] (K x N); Y = relu?(alpha*D + beta*C + row_bias).
// An operand is "MN-major" when its row (A') / column (B') index is the contiguous one.
// ld = element stride of the non-contiguous axis, bs = element stride between batches.
struct TcGemmProblem {
    int M, N, K, batch;
    const float *A, *B;
    int a_mn_major, b_mn_major;
    long long a_ld, b_ld, a_bs, b_bs;
    int a_batched, b_batched;
    float alpha, beta;
    const float *C;
    long long c_si, c_sj, c_sb;
    const float *row_bias;
    const float *residual;   // optional addend with Y's own layout, added before Relu (ignored when C is given)
    int relu;
    float *Y;
    long long y_ld, y_bs;
    // When y_split > 0 the N columns are `y_split`-wide groups laid y_group_stride elements apart in Y
    // (column j lives at (j / y_split) * y_group_stride + j % y_split of its row): the pixels of several
    // NCHW images contracted as one wide GEMM.
    int y_split;
    long long y_group_stride;
};

bool tc_gemm_supports(const TcGemmProblem &g);
int launch_tc_gemm(const TcGemmProblem &g, void *stream);
// Split-K form for small M and a long reduction (tc_gemm_splitk.cu); launch_tc_gemm uses it where it fits.
bool tc_gemm_splitk_fits(const TcGemmProblem &g);
int launch_tc_gemm_splitk(const TcGemmProblem &g, void *stream);

// Address of the device error word of the current device (NULL on failure).
unsigned int *device_status_ptr();

namespace tc_host {
// Launch `kernel` so that it may begin (up to its pdl_wait()) before the previous kernel of the stream
// has finished.  Returns the cudaError_t of the launch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same for a kernel launched as clusters of `cluster_x` CTAs along x (grid.x a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), unsigned cluster_x, dim3 grid, dim3 block, size_t smem,
                                      cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kTmapSwizzleNone = 0, kTmapSwizzle128 = 1, kTmapSwizzle128Atom32 = 2;
bool make_tmap(CUtensorMap *out, const void *base, int rank, const uint64_t *dims, const uint64_t *strides_bytes,
               const uint32_t *box, int swizzle);
int num_sms();
}  // namespace tc_host

}  // namespace onnxb
