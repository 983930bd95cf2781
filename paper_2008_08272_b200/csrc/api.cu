// C-ABI run calls: argument checks, dispatch, launch.  Nothing here allocates
// device memory or synchronises (except onnxb_last_device_status, by contract).
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>

#include "common.h"
#include "tc_common.cuh"
#include "tc_host.h"

using namespace onnxb;

namespace onnxb {
// Error word set by bounded device-side waits that ran out.
__device__ unsigned int g_device_status_word = 0;
unsigned int *device_status_ptr() {
    // per-device cache; the value is the same whichever thread stores it first
    static std::atomic<unsigned int *> ptrs[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    unsigned int *cached = ptrs[dev].load(std::memory_order_acquire);
    if (!cached) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status_word) != cudaSuccess) return nullptr;
        cached = static_cast<unsigned int *>(p);
        ptrs[dev].store(cached, std::memory_order_release);
    }
    return cached;
}

// Copy of the weights rounded to TF32 (nearest).  The GEMM kernel hands its operands to the tensor
// core as they are stored, and the hardware ignores the low 13 mantissa bits (truncation, one-sided);
// rounding the constant operand once keeps its error at 2^-11 per term and zero on average.
// Two arrays in one launch (the second may be empty).
__global__ void round_tf32_copy_kernel(const float4 *__restrict__ in0, float4 *__restrict__ out0, unsigned n0,
                                       const float4 *__restrict__ in1, float4 *__restrict__ out1, unsigned n1) {
    tc::pdl_launch_dependents();
    tc::pdl_wait();
    const unsigned total = n0 + n1;
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const bool first = i < n0;
        const float4 v = __ldg(first ? in0 + i : in1 + (i - n0));
        const float4 r = make_float4(tc::round_tf32(v.x), tc::round_tf32(v.y), tc::round_tf32(v.z), tc::round_tf32(v.w));
        if (first) out0[i] = r;
        else out1[i - n0] = r;
    }
}
// counts are multiples of 4 (the callers' leading dimensions are)
static int launch_round_tf32_copy(const float *in0, float *out0, long long count0, const float *in1, float *out1,
                                  long long count1, void *stream) {
    const unsigned n0 = (unsigned)(count0 / 4), n1 = (unsigned)(count1 / 4);
    const int blocks = (int)std::min<long long>(((long long)n0 + n1 + 255) / 256, 148 * 8);
    const cudaError_t e = tc_host::launch_pdl(round_tf32_copy_kernel, dim3(blocks), dim3(256), 0, (cudaStream_t)stream,
                                              reinterpret_cast<const float4 *>(in0), reinterpret_cast<float4 *>(out0), n0,
                                              reinterpret_cast<const float4 *>(in1), reinterpret_cast<float4 *>(out1), n1);
    count_launch();
    return (int)e;
}

// A 1x1, stride-1, unpadded, ungrouped convolution is one GEMM per image:
// Y[n] (M x HW) = W (M x C) * X[n] (C x HW), with W K-major and X[n] pixel-major.
static TcGemmProblem conv1x1_as_gemm(const ConvGeom &g, const float *X, const float *W, const float *B, float *Y,
                                     const float *R = nullptr) {
    TcGemmProblem t{};
    const long long HW = (long long)g.H * g.W;
    t.M = g.M; t.N = (int)HW; t.K = g.C; t.batch = g.N;
    t.A = W; t.B = X;
    t.a_mn_major = 0; t.b_mn_major = 1;
    t.a_ld = g.C; t.b_ld = HW; t.a_bs = 0; t.b_bs = (long long)g.C * HW;
    t.a_batched = 0; t.b_batched = 1;
    t.alpha = 1.f; t.beta = 0.f; t.C = nullptr;
    t.row_bias = B; t.relu = g.relu; t.residual = R;
    t.Y = Y; t.y_ld = HW; t.y_bs = (long long)g.M * HW;
    return t;
}

bool conv_fits_mma_gemm(const ConvGeom &g) {
    if (!(g.kH == 1 && g.kW == 1 && g.sh == 1 && g.sw == 1 && g.group == 1)) return false;
    if (g.pt || g.pl || g.pb || g.pr) return false;
    if (g.C < 32) return false;              // thin contraction: exact fp32 FMA instead
    return tc_gemm_supports(conv1x1_as_gemm(g, nullptr, nullptr, nullptr, nullptr));
}

// Any other unpadded, ungrouped 1x1 convolution (a stride, or an image whose H*W is not a multiple
// of 4 so that TMA cannot address its channel planes): the pixels it reads are first gathered into
// a dense copy Xg[n][c][pitch] (pitch = P*Q rounded up to 4), rounded to TF32 on the way; then the
// same GEMM runs on the copy.
// Two layouts of the copy.  Images whose P*Q is a multiple of 4 and not small keep one GEMM per image
// (Xg[n][c][P*Q], output written by TMA).  Small or oddly sized images are merged: Xg[c][n*P*Q + j]
// with the row pitch rounded up to 4, so that ONE wide GEMM Y' (M x N*P*Q) = W (M x C) * Xg serves all
// images and the weights are streamed once per pixel tile instead of once per image; the epilogue then
// scatters column n*P*Q + j to Y[n][m][j].
static bool gather_merged(const ConvGeom &g) {
    const long long PQ = (long long)g.P * g.Q;
    return PQ % 4 != 0 || PQ < 128;
}
static long long gather_pitch(const ConvGeom &g) {
    const long long PQ = (long long)g.P * g.Q;
    return gather_merged(g) ? (PQ * g.N + 3) / 4 * 4 : PQ;
}

static TcGemmProblem conv1x1_gathered_as_gemm(const ConvGeom &g, const float *Xg, const float *W, const float *B,
                                              float *Y, const float *R = nullptr) {
    TcGemmProblem t{};
    const long long PQ = (long long)g.P * g.Q, pitch = gather_pitch(g);
    const bool merged = gather_merged(g);
    t.M = g.M; t.K = g.C;
    t.A = W; t.B = Xg;
    t.a_mn_major = 0; t.b_mn_major = 1;
    t.a_ld = g.C; t.b_ld = pitch; t.a_bs = 0; t.a_batched = 0;
    t.alpha = 1.f; t.beta = 0.f; t.C = nullptr;
    t.row_bias = B; t.relu = g.relu; t.residual = R;
    t.Y = Y; t.y_ld = PQ;
    if (merged) {
        t.N = (int)(PQ * g.N); t.batch = 1; t.b_bs = 0; t.b_batched = 0; t.y_bs = 0;
        t.y_split = (int)PQ; t.y_group_stride = (long long)g.M * PQ;
    } else {
        t.N = (int)PQ; t.batch = g.N; t.b_bs = (long long)g.C * pitch; t.b_batched = 1;
        t.y_bs = (long long)g.M * PQ;
        t.y_split = 0; t.y_group_stride = 0;
    }
    return t;
}

bool conv_fits_mma_gather_gemm(const ConvGeom &g) {
    if (!(g.kH == 1 && g.kW == 1 && g.group == 1)) return false;
    if (g.pt || g.pl || g.pb || g.pr) return false;
    if (g.C < 32) return false;
    if ((long long)g.N * g.C * ((long long)g.P * g.Q + 4) > 2147483647LL) return false;
    return tc_gemm_supports(conv1x1_gathered_as_gemm(g, nullptr, nullptr, nullptr, nullptr));
}

size_t conv_gather_workspace_bytes(const ConvGeom &g) {
    return (size_t)g.C * gather_pitch(g) * 4 * (gather_merged(g) ? 1 : g.N);
}

}  // namespace onnxb

static inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// w_copy (gather family only): a TF32-rounded copy of W made earlier by onnx_conv2d_prepack; the workspace
// then only has to hold the gathered input.
static onnxb_status conv2d_run_impl(onnxb_conv2d_desc_t d, const float *X, const float *W, const float *B,
                                    const float *R, float *Y, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream, int phase = kTcConvPackAndRun, const float *w_copy = nullptr) {
    const bool pack_only = phase == kTcConvPackOnly;
    if (!d || !W || (!pack_only && (!X || !Y))) return ONNXB_ERR_NULL;
    if (misaligned(R)) return ONNXB_ERR_UNSUPPORTED;
    if (!pack_only && (d->g.has_bias != 0) != (B != nullptr)) return ONNXB_ERR_NULL;
    const size_t wr_bytes = (size_t)d->g.M * d->g.C * 4;           // the gather family's rounded weights
    size_t need = d->workspace_bytes;
    if (d->family == ONNXB_KERNEL_MMA_GATHER_GEMM) need = pack_only ? wr_bytes : w_copy ? need - wr_bytes : need;
    if (need > 0 && (!workspace || workspace_bytes < need)) return ONNXB_ERR_WORKSPACE;
    if (misaligned(X) || misaligned(W) || misaligned(B) || misaligned(Y) || misaligned(workspace))
        return ONNXB_ERR_UNSUPPORTED;

    int err;
    switch (d->family) {
        case ONNXB_KERNEL_SIMT_DEPTHWISE:
            err = launch_simt_depthwise(d->g, X, W, B, R, Y, cuda_stream);
            break;
        case ONNXB_KERNEL_SIMT_DIRECT:
            err = launch_simt_conv(d->g, X, W, B, R, Y, cuda_stream);
            break;
        case ONNXB_KERNEL_MMA_GEMM: {
            // the workspace holds W rounded to TF32 (made here, or earlier by onnx_conv2d_prepack)
            float *Wr = static_cast<float *>(workspace);
            err = 0;
            if (phase != kTcConvRunOnly) err = launch_round_tf32_copy(W, Wr, (long long)d->g.M * d->g.C, nullptr, nullptr, 0, cuda_stream);
            if (err == 0 && phase != kTcConvPackOnly) err = launch_tc_gemm(conv1x1_as_gemm(d->g, X, Wr, B, Y, R), cuda_stream);
            break;
        }
        case ONNXB_KERNEL_MMA_GATHER_GEMM: {
            // workspace: [W rounded to TF32][gathered input]; with a copy of W made ahead, the gathered input alone
            float *ws = static_cast<float *>(workspace);
            const float *Wr = w_copy ? w_copy : ws;
            float *Xg = w_copy ? ws : ws + (size_t)d->g.M * d->g.C;
            err = 0;
            if (!w_copy) err = launch_round_tf32_copy(W, ws, (long long)d->g.M * d->g.C, nullptr, nullptr, 0, cuda_stream);
            if (pack_only) break;
            if (err == 0) err = launch_gather1x1(d->g, X, Xg, gather_pitch(d->g), gather_merged(d->g), cuda_stream);
            if (err == 0) err = launch_tc_gemm(conv1x1_gathered_as_gemm(d->g, Xg, Wr, B, Y, R), cuda_stream);
            break;
        }
        case ONNXB_KERNEL_MMA_IMPLICIT:
            err = launch_tc_conv(d->plan, X, W, B, R, Y, workspace, cuda_stream, phase);
            break;
        default:
            return ONNXB_ERR_UNSUPPORTED;
    }
    return err == 0 ? ONNXB_OK : ONNXB_ERR_CUDA;
}

extern "C" onnxb_status onnx_conv2d_run(onnxb_conv2d_desc_t d, const float *X, const float *W,
                                        const float *B, float *Y, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream) {
    return conv2d_run_impl(d, X, W, B, nullptr, Y, workspace, workspace_bytes, cuda_stream);
}

// Conv followed by Add (a residual connection) and the descriptor's Relu, in one pass: the single-use
// producer/consumer fusion of Sec. 3.4.3 applied to Conv -> Add -> Relu.
extern "C" onnxb_status onnx_conv2d_add_run(onnxb_conv2d_desc_t d, const float *X, const float *W, const float *B,
                                            const float *R, float *Y, void *workspace, size_t workspace_bytes,
                                            void *cuda_stream) {
    if (!R) return ONNXB_ERR_NULL;
    return conv2d_run_impl(d, X, W, B, R, Y, workspace, workspace_bytes, cuda_stream);
}

// Weights known ahead of the run (an inference graph's constants, Sec. 3.4.4): the implicit-GEMM
// kernel's packing step done once, and run calls that take the packed copy instead of redoing it.
// Which kernel families keep a derived copy of W in their scratch (packed and/or rounded to TF32).
static bool family_has_weight_copy(int family) {
    return family == ONNXB_KERNEL_MMA_IMPLICIT || family == ONNXB_KERNEL_MMA_GEMM || family == ONNXB_KERNEL_MMA_GATHER_GEMM;
}

extern "C" onnxb_status onnx_conv2d_prepack(onnxb_conv2d_desc_t d, const float *W, void *packed, size_t packed_bytes,
                                            void *cuda_stream) {
    if (!d || !W) return ONNXB_ERR_NULL;
    if (!family_has_weight_copy(d->family)) return ONNXB_OK;              // the other kernels read W as it is
    // (the gather family's copy is only the rounded W, the leading part of its workspace)
    const size_t need = d->family == ONNXB_KERNEL_MMA_GATHER_GEMM ? (size_t)d->g.M * d->g.C * 4 : d->workspace_bytes;
    if (!packed || packed_bytes < need) return ONNXB_ERR_WORKSPACE;
    return conv2d_run_impl(d, nullptr, W, nullptr, nullptr, nullptr, packed, packed_bytes, cuda_stream, kTcConvPackOnly);
}

extern "C" onnxb_status onnx_conv2d_run_prepacked(onnxb_conv2d_desc_t d, const float *X, const float *W,
                                                  const void *packed, const float *B, const float *R, float *Y,
                                                  void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!d) return ONNXB_ERR_NULL;
    if (!family_has_weight_copy(d->family))
        return conv2d_run_impl(d, X, W, B, R, Y, workspace, workspace_bytes, cuda_stream);
    if (!packed) return ONNXB_ERR_NULL;
    if (d->family == ONNXB_KERNEL_MMA_GATHER_GEMM)      // the copy of W from `packed`, the gathered input in the workspace
        return conv2d_run_impl(d, X, W, B, R, Y, workspace, workspace_bytes, cuda_stream, kTcConvRunOnly,
                               static_cast<const float *>(packed));
    // the packed copy stands in for the workspace; its size was checked when it was made
    return conv2d_run_impl(d, X, W, B, R, Y, const_cast<void *>(packed), d->workspace_bytes, cuda_stream, kTcConvRunOnly);
}

// ONNX Gemm on the tensor cores reads rounded copies of both operands: the tensor core would otherwise
// truncate them (one-sided, up to 2^-10 per operand), which leaves the stated error bound for operands
// of one sign.  Both copies live in the workspace: A' first, then B'.
static bool gemm_tc_eligible(int transA, int transB, int64_t M, int64_t N, int64_t K) {
    if (K < 32) return false;                       // thin contraction: exact fp32 FMA instead
    const int64_t a_ld = transA ? M : K, b_ld = transB ? K : N;
    return a_ld % 4 == 0 && b_ld % 4 == 0;          // tensor-map strides are multiples of 16 bytes
}

extern "C" size_t onnx_gemm_workspace_bytes(int transA, int transB, int64_t M, int64_t N, int64_t K) {
    if (M < 1 || N < 1 || K < 1) return 0;
    return gemm_tc_eligible(transA, transB, M, N, K) ? (size_t)(M * K + K * N) * 4 : 0;
}

extern "C" onnxb_status onnx_gemm_run(int transA, int transB, float alpha, float beta, int64_t M, int64_t N,
                                      int64_t K, const float *A, const float *B, const float *C, int c_rank,
                                      const int64_t *c_dims, int fuse_relu, float *Y, void *workspace,
                                      size_t workspace_bytes, void *cuda_stream) {
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

    // Tensor-core path unless the contraction is thin or an operand cannot be described to TMA.
    TcGemmProblem t{};
    t.M = p.M; t.N = p.N; t.K = p.K; t.batch = 1;
    t.A = A; t.B = B;
    t.a_mn_major = p.transA; t.a_ld = p.transA ? p.M : p.K;
    t.b_mn_major = !p.transB; t.b_ld = p.transB ? p.K : p.N;
    t.alpha = alpha; t.beta = beta; t.C = C; t.c_si = p.c_stride_i; t.c_sj = p.c_stride_j; t.c_sb = 0;
    t.row_bias = nullptr; t.relu = p.relu;
    t.Y = Y; t.y_ld = p.N; t.y_bs = 0;
    const int forced = kernel_override();
    const bool forced_tc = forced == ONNXB_KERNEL_MMA_GEMM || forced == ONNXB_KERNEL_MMA_IMPLICIT;
    const bool eligible = gemm_tc_eligible(transA, transB, M, N, K) && tc_gemm_supports(t);
    int err;
    if (eligible && (forced_tc || forced < 0)) {
        const size_t need = onnx_gemm_workspace_bytes(transA, transB, M, N, K);
        if (!workspace || workspace_bytes < need) return ONNXB_ERR_WORKSPACE;
        if (tc_gemm_splitk_fits(t)) {
            // few tiles and a long reduction: the split-K kernel rounds its operands itself
            err = launch_tc_gemm(t, cuda_stream);
        } else {
            float *Ar = static_cast<float *>(workspace), *Br = Ar + M * K;
            err = launch_round_tf32_copy(A, Ar, M * K, B, Br, K * N, cuda_stream);
            t.A = Ar; t.B = Br;
            if (err == 0) err = launch_tc_gemm(t, cuda_stream);
        }
    } else if (forced_tc) {
        return ONNXB_ERR_UNSUPPORTED;
    } else {
        err = launch_simt_gemm(p, A, B, C, Y, cuda_stream);
    }
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

// MatMul followed by Add, as the graph rewriting of Sec. 3.4.3 fuses them: Gemm with no transposition
// and unit scale factors.
extern "C" onnxb_status onnx_matmul_add_run(int64_t M, int64_t N, int64_t K, const float *A, const float *B,
                                            const float *C, int c_rank, const int64_t *c_dims, int fuse_relu,
                                            float *Y, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return onnx_gemm_run(0, 0, 1.0f, 1.0f, M, N, K, A, B, C, c_rank, c_dims, fuse_relu, Y, workspace, workspace_bytes,
                         cuda_stream);
}
