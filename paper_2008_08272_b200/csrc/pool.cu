// ONNX MaxPool (2-D, NCHW) and GlobalAveragePool: the pooling operators of the two models the
// paper runs (Sec. 4.1 lists pooling among the lowered operators; Sec. 4.2: MNIST has a MaxPool,
// ResNet50 a 3x3 stride-2 MaxPool after the stem and a global average pool before the classifier).
// Both are pure data movement: 0.1-1 flop per byte, bound by HBM.
#include <cuda_runtime.h>

#include <cfloat>

#include "common.h"
#include "tc_conv_plan.h"

namespace onnxb {
namespace {

// MaxPool: a thread owns one output row segment of four consecutive columns of one (n, c) plane and
// walks the kH input rows it needs once; neighbouring threads' overlapping reads are served by L1.
// Positions outside the image do not take part (the padding value of ONNX MaxPool is minus infinity).
__global__ void __launch_bounds__(256)
maxpool2d_kernel(const float *__restrict__ X, float *__restrict__ Y, int H, int W, int P, int Q, int kH, int kW,
                 int pt, int pl, int sh, int sw, unsigned items, unsigned Q4, ConvDivisor dv_Q4, ConvDivisor dv_P) {
    const unsigned i = blockIdx.x * 256u + threadIdx.x;
    if (i >= items) return;
    const unsigned t = (unsigned)conv_fdiv((int)i, (int)Q4, dv_Q4), q4 = i - t * Q4;
    const unsigned plane = (unsigned)conv_fdiv((int)t, P, dv_P), p = t - plane * (unsigned)P;
    const int q0 = (int)q4 * 4;
    const float *xp = X + (size_t)plane * H * W;
    float best[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    const int h0 = (int)p * sh - pt;
    for (int r = 0; r < kH; ++r) {
        const int h = h0 + r;
        if ((unsigned)h >= (unsigned)H) continue;
        const float *row = xp + (size_t)h * W;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w0 = (q0 + j) * sw - pl;
            for (int s = 0; s < kW; ++s) {
                const int w = w0 + s;
                if ((unsigned)w < (unsigned)W) best[j] = fmaxf(best[j], __ldg(row + w));
            }
        }
    }
    float *yp = Y + ((size_t)plane * P + p) * Q + q0;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (q0 + j < Q) yp[j] = best[j];
}

// The ResNet-50 pool: 3x3 window, stride 2, one row/column of padding in front (any amount behind),
// even width a multiple of 8.  A thread owns 4 output columns x 2 output rows: the five input rows they
// need are read once each, as two aligned 16-byte loads plus the column in front.
__global__ void __launch_bounds__(256)
maxpool_3x3s2_kernel(const float *__restrict__ X, float *__restrict__ Y, int H, int W, int P, int Q, unsigned items,
                     unsigned Q4, unsigned P2, ConvDivisor dv_Q4, ConvDivisor dv_P2) {
    const unsigned i = blockIdx.x * 256u + threadIdx.x;
    if (i >= items) return;
    const unsigned t = (unsigned)conv_fdiv((int)i, (int)Q4, dv_Q4), q4 = i - t * Q4;
    const unsigned plane = (unsigned)conv_fdiv((int)t, (int)P2, dv_P2), p2 = t - plane * P2;
    const int p0 = (int)p2 * 2, q0 = (int)q4 * 4, w0 = q0 * 2;          // first input column of the strip is w0 - 1
    const float *xp = X + (size_t)plane * H * W;
    float top[4], bot[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) top[j] = bot[j] = -INFINITY;
#pragma unroll
    for (int rr = 0; rr < 5; ++rr) {
        const int h = p0 * 2 - 1 + rr;
        if ((unsigned)h >= (unsigned)H) continue;
        const float *row = xp + (size_t)h * W + w0;
        const float4 a = __ldg(reinterpret_cast<const float4 *>(row));
        const float4 b = w0 + 4 < W ? __ldg(reinterpret_cast<const float4 *>(row + 4)) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        const float l = w0 > 0 ? __ldg(row - 1) : -INFINITY;
        float m[4];                                                      // window maxima of this row for the 4 outputs
        m[0] = fmaxf(fmaxf(l, a.x), a.y);
        m[1] = fmaxf(fmaxf(a.y, a.z), a.w);
        m[2] = fmaxf(fmaxf(a.w, b.x), b.y);
        m[3] = fmaxf(fmaxf(b.y, b.z), b.w);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (rr < 3) top[j] = fmaxf(top[j], m[j]);
            if (rr >= 2) bot[j] = fmaxf(bot[j], m[j]);
        }
    }
    float *yp = Y + ((size_t)plane * P + p0) * Q + q0;
    if (q0 + 3 < Q) {
        *reinterpret_cast<float4 *>(yp) = make_float4(top[0], top[1], top[2], top[3]);
        if (p0 + 1 < P) *reinterpret_cast<float4 *>(yp + Q) = make_float4(bot[0], bot[1], bot[2], bot[3]);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (q0 + j < Q) {
                yp[j] = top[j];
                if (p0 + 1 < P) yp[Q + j] = bot[j];
            }
    }
}

// GlobalAveragePool: TPP threads per (n, c) plane (8 for small planes, 32 otherwise) striding over it,
// partial sums in fp32, then a shuffle tree inside the group.
template <int TPP>
__global__ void __launch_bounds__(256)
global_average_pool_kernel(const float *__restrict__ X, float *__restrict__ Y, unsigned planes, unsigned HW, float inv_hw) {
    const unsigned gid = (blockIdx.x * 256u + threadIdx.x) / TPP, sub = threadIdx.x % TPP;
    float acc = 0.f;
    if (gid < planes) {
        const float *xp = X + (size_t)gid * HW;
        for (unsigned k = sub; k < HW; k += TPP) acc += __ldg(xp + k);
    }
#pragma unroll
    for (int o = TPP / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (gid < planes && sub == 0) Y[gid] = acc * inv_hw;
}

bool pool_shape(const int64_t *x, const int64_t *k, const int64_t *pads, const int64_t *st, int64_t *y) {
    if (!x || !k) return false;
    const int64_t pt = pads ? pads[0] : 0, pl = pads ? pads[1] : 0, pb = pads ? pads[2] : 0, pr = pads ? pads[3] : 0;
    const int64_t sh = st && st[0] ? st[0] : 1, sw = st && st[1] ? st[1] : 1;
    if (x[0] < 1 || x[1] < 1 || x[2] < 1 || x[3] < 1 || k[0] < 1 || k[1] < 1 || sh < 1 || sw < 1) return false;
    if (pt < 0 || pl < 0 || pb < 0 || pr < 0) return false;
    if (pt >= k[0] || pb >= k[0] || pl >= k[1] || pr >= k[1]) return false;     // a window made of padding only
    if (x[2] + pt + pb < k[0] || x[3] + pl + pr < k[1]) return false;
    y[0] = x[0];
    y[1] = x[1];
    y[2] = (x[2] + pt + pb - k[0]) / sh + 1;
    y[3] = (x[3] + pl + pr - k[1]) / sw + 1;
    return true;
}

}  // namespace
}  // namespace onnxb

using namespace onnxb;

extern "C" onnxb_status onnx_maxpool2d_shape(const int64_t x_dims[4], const int64_t kernel_shape[2],
                                             const int64_t pads[4], const int64_t strides[2], int64_t y_dims[4]) {
    if (!x_dims || !kernel_shape || !y_dims) return ONNXB_ERR_NULL;
    return pool_shape(x_dims, kernel_shape, pads, strides, y_dims) ? ONNXB_OK : ONNXB_ERR_SHAPE;
}

extern "C" onnxb_status onnx_maxpool2d_run(const int64_t x_dims[4], const int64_t kernel_shape[2],
                                           const int64_t pads[4], const int64_t strides[2], const float *X, float *Y,
                                           void *cuda_stream) {
    if (!x_dims || !kernel_shape || !X || !Y) return ONNXB_ERR_NULL;
    int64_t y[4];
    if (!pool_shape(x_dims, kernel_shape, pads, strides, y)) return ONNXB_ERR_SHAPE;
    const int64_t lim = 2147483647LL;
    if (x_dims[0] * x_dims[1] * x_dims[2] * x_dims[3] > lim || kernel_shape[0] > 1024 || kernel_shape[1] > 1024)
        return ONNXB_ERR_UNSUPPORTED;
    const int P = (int)y[2], Q = (int)y[3];
    const int64_t pt0 = pads ? pads[0] : 0, pl0 = pads ? pads[1] : 0;
    const int64_t sh0 = strides && strides[0] ? strides[0] : 1, sw0 = strides && strides[1] ? strides[1] : 1;
    if (kernel_shape[0] == 3 && kernel_shape[1] == 3 && sh0 == 2 && sw0 == 2 && pt0 == 1 && pl0 == 1 &&
        x_dims[3] % 8 == 0 && Q * 2 == x_dims[3] && (reinterpret_cast<uintptr_t>(X) & 15) == 0 &&
        (reinterpret_cast<uintptr_t>(Y) & 15) == 0 && Q % 4 == 0) {
        const unsigned Q4s = (unsigned)(Q / 4), P2 = (unsigned)((P + 1) / 2);
        const int64_t n_items = y[0] * y[1] * P2 * Q4s;
        if (n_items > lim - 256) return ONNXB_ERR_UNSUPPORTED;
        maxpool_3x3s2_kernel<<<(unsigned)((n_items + 255) / 256), 256, 0, (cudaStream_t)cuda_stream>>>(
            X, Y, (int)x_dims[2], (int)x_dims[3], P, Q, (unsigned)n_items, Q4s, P2, conv_divisor((int)Q4s),
            conv_divisor((int)P2));
        count_launch();
        return cudaGetLastError() == cudaSuccess ? ONNXB_OK : ONNXB_ERR_CUDA;
    }
    const unsigned Q4 = (unsigned)((Q + 3) / 4);
    const int64_t items = y[0] * y[1] * P * Q4;
    if (items > lim - 256) return ONNXB_ERR_UNSUPPORTED;
    const unsigned blocks = (unsigned)((items + 255) / 256);
    maxpool2d_kernel<<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(
        X, Y, (int)x_dims[2], (int)x_dims[3], P, Q, (int)kernel_shape[0], (int)kernel_shape[1], pads ? (int)pads[0] : 0,
        pads ? (int)pads[1] : 0, strides && strides[0] ? (int)strides[0] : 1, strides && strides[1] ? (int)strides[1] : 1,
        (unsigned)items, Q4, conv_divisor((int)Q4), conv_divisor(P));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? ONNXB_OK : ONNXB_ERR_CUDA;
}

extern "C" onnxb_status onnx_global_average_pool_run(const int64_t x_dims[4], const float *X, float *Y,
                                                     void *cuda_stream) {
    if (!x_dims || !X || !Y) return ONNXB_ERR_NULL;
    if (x_dims[0] < 1 || x_dims[1] < 1 || x_dims[2] < 1 || x_dims[3] < 1) return ONNXB_ERR_SHAPE;
    const int64_t planes = x_dims[0] * x_dims[1], hw = x_dims[2] * x_dims[3];
    if (planes > (1LL << 26) || hw > (1LL << 30) || planes * hw > 2147483647LL * 4) return ONNXB_ERR_UNSUPPORTED;
    if (hw <= 128) {
        const unsigned blocks = (unsigned)((planes * 8 + 255) / 256);
        global_average_pool_kernel<8><<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(X, Y, (unsigned)planes, (unsigned)hw,
                                                                                   1.0f / (float)hw);
    } else {
        const unsigned blocks = (unsigned)((planes * 32 + 255) / 256);
        global_average_pool_kernel<32><<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(X, Y, (unsigned)planes, (unsigned)hw,
                                                                                    1.0f / (float)hw);
    }
    count_launch();
    return cudaGetLastError() == cudaSuccess ? ONNXB_OK : ONNXB_ERR_CUDA;
}
