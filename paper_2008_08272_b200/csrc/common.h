// Internal declarations shared by the translation units of libonnx_b200.
#pragma once
#include <atomic>
#include <cstddef>
#include <cstdint>

#include "onnx_b200.h"
#include "tc_conv_plan.h"

namespace onnxb {

// A convolution problem with every ONNX default and auto_pad already resolved.
struct ConvGeom {
    int N, C, H, W;          // input
    int M, Cg, kH, kW;       // weights: M output channels, Cg = C/group input channels each
    int P, Q;                // output spatial size
    int pt, pl, pb, pr;      // resolved pads (h_begin, w_begin, h_end, w_end)
    int sh, sw, dh, dw;
    int group, Mg;           // Mg = M/group
    int has_bias, relu;
};

}  // namespace onnxb

struct onnxb_conv2d_desc_s {
    onnxb::ConvGeom g;
    int family;              // onnxb_kernel_family
    onnxb::TcConvPlan plan;  // valid when family == ONNXB_KERNEL_MMA_IMPLICIT
    size_t workspace_bytes;
    int64_t y_dims[4];
    int64_t pads[4];
};

namespace onnxb {

extern std::atomic<uint64_t> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int kernel_override();   // -1 = automatic

// SIMT family (simt_conv.cu / simt_gemm.cu).  All return a cudaError_t as int.
// R (everywhere below): optional addend with Y's shape, added before Relu (a residual connection); may be NULL.
int launch_simt_conv(const ConvGeom &g, const float *X, const float *W, const float *B, const float *R, float *Y,
                     void *stream);
int launch_simt_depthwise(const ConvGeom &g, const float *X, const float *W, const float *B, const float *R, float *Y,
                          void *stream);
bool simt_depthwise_supports(const ConvGeom &g);
bool conv_fits_mma_gemm(const ConvGeom &g);
bool conv_fits_mma_gather_gemm(const ConvGeom &g);   // other unpadded 1x1: gather the pixels read, then the same GEMM
size_t conv_gather_workspace_bytes(const ConvGeom &g);
int launch_gather1x1(const ConvGeom &g, const float *X, float *Xg, long long pitch, bool merged, void *stream);
// implicit-GEMM tensor-core convolution (tc_conv.cu)
bool tc_conv_plan(const ConvGeom &g, TcConvPlan &plan, bool forced = false);
size_t tc_conv_workspace_bytes(const TcConvPlan &plan);
// phase: both steps (pack the weights into the workspace, then convolve), or one of them alone
constexpr int kTcConvPackAndRun = 0, kTcConvPackOnly = 1, kTcConvRunOnly = 2;
int launch_tc_conv(const TcConvPlan &plan, const float *X, const float *W, const float *B, const float *R, float *Y,
                   void *workspace, void *stream, int phase = kTcConvPackAndRun);   // 1x1 stride-1 convolution expressible as a batched TMA GEMM

struct GemmProblem {
    int M, N, K;
    int transA, transB;
    float alpha, beta;
    long long c_stride_i, c_stride_j;   // element strides of C along i and j (0 = broadcast)
    int relu;
};
int launch_simt_gemm(const GemmProblem &p, const float *A, const float *B, const float *C, float *Y,
                     void *stream);

}  // namespace onnxb
