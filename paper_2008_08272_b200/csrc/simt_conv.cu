// SIMT (fp32 FMA) convolution kernels: the path for contractions too thin for
// the tensor cores (few input channels per group, depthwise) and the general
// fallback that accepts every attribute combination of ONNX Conv (Sec. 4.1).
#include <cuda_runtime.h>

#include <algorithm>

#include "common.h"
#include "tc_common.cuh"

namespace onnxb {

namespace {

constexpr int kDirectThreads = 128;   // one output pixel per thread
constexpr int kDirectChunk = 256;     // reduction terms staged in shared memory per pass

// Direct convolution.  A block owns 128 consecutive output pixels of one image
// and MT consecutive output channels of one group; each thread keeps MT
// accumulators, so every input value loaded is used MT times.  The reduction
// index k = (c*kH + r)*kW + s is walked in chunks whose weights sit in shared
// memory (all threads read the same weight: a broadcast).
template <int MT>
__global__ void __launch_bounds__(kDirectThreads)
conv2d_direct_kernel(const ConvGeom g, const float *__restrict__ X, const float *__restrict__ W,
                     const float *__restrict__ B, const float *__restrict__ R, float *__restrict__ Y, int pixel_tiles,
                     int m_tiles_per_group) {
    __shared__ float wsm[MT * kDirectChunk];

    const int tile = blockIdx.x % pixel_tiles;
    const int n = blockIdx.x / pixel_tiles;
    const int PQ = g.P * g.Q;
    const int pix = tile * kDirectThreads + threadIdx.x;
    const bool live = pix < PQ;
    const int p = live ? pix / g.Q : 0;
    const int q = live ? pix % g.Q : 0;
    const int ih0 = p * g.sh - g.pt;
    const int iw0 = q * g.sw - g.pl;
    const int taps = g.kH * g.kW;
    const int Kred = g.Cg * taps;

    for (int mt = blockIdx.y; mt < m_tiles_per_group * g.group; mt += gridDim.y) {
        const int grp = mt / m_tiles_per_group;
        const int m0 = grp * g.Mg + (mt % m_tiles_per_group) * MT;
        const int m_end = (grp + 1) * g.Mg;
        const float *xg = X + ((size_t)n * g.C + (size_t)grp * g.Cg) * g.H * g.W;

        float acc[MT];
#pragma unroll
        for (int j = 0; j < MT; ++j) acc[j] = 0.f;

        for (int k0 = 0; k0 < Kred; k0 += kDirectChunk) {
            const int len = min(kDirectChunk, Kred - k0);
            __syncthreads();
            for (int idx = threadIdx.x; idx < MT * len; idx += kDirectThreads) {
                const int j = idx / len, kk = idx - j * len;
                wsm[j * kDirectChunk + kk] = (m0 + j < m_end) ? W[(size_t)(m0 + j) * Kred + k0 + kk] : 0.f;
            }
            __syncthreads();
            if (live) {
                int c = k0 / taps;
                int rs = k0 - c * taps;
                int r = rs / g.kW;
                int s = rs - r * g.kW;
                for (int kk = 0; kk < len; ++kk) {
                    const int ih = ih0 + r * g.dh;
                    const int iw = iw0 + s * g.dw;
                    float x = 0.f;
                    if ((unsigned)ih < (unsigned)g.H && (unsigned)iw < (unsigned)g.W)
                        x = __ldg(xg + ((size_t)c * g.H + ih) * g.W + iw);
#pragma unroll
                    for (int j = 0; j < MT; ++j) acc[j] = fmaf(x, wsm[j * kDirectChunk + kk], acc[j]);
                    if (++s == g.kW) {
                        s = 0;
                        if (++r == g.kH) {
                            r = 0;
                            ++c;
                        }
                    }
                }
            }
        }
        if (live) {
#pragma unroll
            for (int j = 0; j < MT; ++j) {
                const int m = m0 + j;
                if (m < m_end) {
                    float v = acc[j] + (B ? __ldg(B + m) : 0.f);
                    const size_t yi = ((size_t)n * g.M + m) * PQ + pix;
                    if (R) v += __ldg(R + yi);              // residual addend at Y's own position
                    if (g.relu) v = v > 0.f ? v : 0.f;
                    Y[yi] = v;
                }
            }
        }
    }
}

// Depthwise convolution (group == C == M): purely HBM-bound, 2*kH*kW flops per
// output.  A block stages the input window of a 32 x 32 output tile of one
// (image, channel) plane in shared memory with coalesced row loads (zeros
// outside the image); each of its 256 threads then produces a column strip of
// four vertically adjacent outputs, so the rows of the window shared by the
// four outputs are read from shared memory once per tap column.
constexpr int kDwTP = 32, kDwTQ = 32, kDwRows = 4, kDwThreads = kDwTQ * (kDwTP / kDwRows);

__global__ void __launch_bounds__(kDwThreads)
conv2d_depthwise_kernel(const ConvGeom g, const float *__restrict__ X, const float *__restrict__ W,
                        const float *__restrict__ B, const float *__restrict__ R, float *__restrict__ Y, int q_tiles,
                        int p_tiles,
                        int in_rows, int in_cols, int pitch) {
    extern __shared__ float tile[];           // [in_rows][pitch] then weights [kH*kW]
    float *wsm = tile + in_rows * pitch;

    int bid = blockIdx.x;
    const int qt = bid % q_tiles; bid /= q_tiles;
    const int pt_ = bid % p_tiles; bid /= p_tiles;
    const int plane = bid;                    // n * C + c
    const int c = plane % g.C;
    const int p0 = pt_ * kDwTP, q0 = qt * kDwTQ;
    const int ih0 = p0 * g.sh - g.pt, iw0 = q0 * g.sw - g.pl;
    const float *xp = X + (size_t)plane * g.H * g.W;

    const int taps = g.kH * g.kW;
    for (int i = threadIdx.x; i < taps; i += kDwThreads) wsm[i] = W[(size_t)c * taps + i];
    // window rows actually needed by this tile (fewer at the bottom edge of the image)
    const int rows_out = min(kDwTP, g.P - p0);
    const int rows_in = min(in_rows, (rows_out - 1) * g.sh + (g.kH - 1) * g.dh + 1);
    for (int i = threadIdx.x; i < rows_in * in_cols; i += kDwThreads) {
        const int rr = i / in_cols, cc = i - rr * in_cols;
        const int ih = ih0 + rr, iw = iw0 + cc;
        float v = 0.f;
        if ((unsigned)ih < (unsigned)g.H && (unsigned)iw < (unsigned)g.W) v = __ldg(xp + (size_t)ih * g.W + iw);
        tile[rr * pitch + cc] = v;
    }
    __syncthreads();

    const int tq = threadIdx.x % kDwTQ, tp = (threadIdx.x / kDwTQ) * kDwRows;
    const int q = q0 + tq;
    if (q >= g.Q || p0 + tp >= g.P) return;
    float acc[kDwRows];
#pragma unroll
    for (int k = 0; k < kDwRows; ++k) acc[k] = 0.f;
    for (int s = 0; s < g.kW; ++s) {
        const float *col = tile + tq * g.sw + s * g.dw;
        for (int r = 0; r < g.kH; ++r) {
            const float w = wsm[r * g.kW + s];
#pragma unroll
            for (int k = 0; k < kDwRows; ++k)
                if (tp + k < rows_out) acc[k] = fmaf(col[((tp + k) * g.sh + r * g.dh) * pitch], w, acc[k]);
        }
    }
    const float bias = B ? __ldg(B + c) : 0.f;
#pragma unroll
    for (int k = 0; k < kDwRows; ++k) {
        const int p = p0 + tp + k;
        if (p < g.P) {
            float v = acc[k] + bias;
            const size_t yi = ((size_t)plane * g.P + p) * g.Q + q;
            if (R) v += __ldg(R + yi);
            if (g.relu) v = v > 0.f ? v : 0.f;
            Y[yi] = v;
        }
    }
}

// Gather for strided / oddly sized 1x1 convolutions, values rounded to TF32 (nearest, ties away):
//   merged:    Xg[c][n*P*Q + p*Q + q] = X[n][c][p*sh][q*sw], rows padded with zeros to the pitch;
//   per image: Xg[n][c][p*Q + q]      (pitch = P*Q).
__device__ __forceinline__ float gather_round(float v) {
    return __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xFFFFE000u);
}

__global__ void __launch_bounds__(256)
gather1x1_kernel(const float *__restrict__ X, float *__restrict__ Xg, unsigned total, unsigned pitch, unsigned NPQ,
                 unsigned PQ, unsigned Q, unsigned C, unsigned HW, unsigned rowstep, unsigned sw, int merged,
                 const ConvDivisor dv_pitch, const ConvDivisor dv_PQ, const ConvDivisor dv_Q) {
    tc::pdl_launch_dependents();
    // the three divisions per element are multiply-and-shift by constants the host prepares
    for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < total; i += gridDim.x * 256u) {
        const unsigned row = (unsigned)conv_fdiv((int)i, (int)pitch, dv_pitch);   // merged: channel; per image: n*C + c
        const unsigned j = i - row * pitch;
        float v = 0.f;
        if (j < NPQ) {
            unsigned plane, r;
            if (merged) {
                const unsigned n = (unsigned)conv_fdiv((int)j, (int)PQ, dv_PQ);
                r = j - n * PQ;
                plane = n * C + row;
            } else {
                r = j;
                plane = row;
            }
            const unsigned p = (unsigned)conv_fdiv((int)r, (int)Q, dv_Q), q = r - p * Q;
            v = gather_round(__ldg(X + (size_t)plane * HW + p * rowstep + q * sw));
        }
        Xg[i] = v;
    }
}

// Any layout whose pitch is a multiple of four (both layouts have one): four consecutive outputs per
// thread, indices divided once and then stepped, four independent scalar loads, one 16-byte store.
__global__ void __launch_bounds__(256)
gather1x1_quad_kernel(const float *__restrict__ X, float4 *__restrict__ Xg4, unsigned total4, unsigned pitch,
                      unsigned NPQ, unsigned PQ, unsigned Q, unsigned C, unsigned HW, unsigned rowstep, unsigned sw,
                      int merged, const ConvDivisor dv_pitch, const ConvDivisor dv_PQ, const ConvDivisor dv_Q) {
    tc::pdl_launch_dependents();
    for (unsigned i4 = blockIdx.x * 256u + threadIdx.x; i4 < total4; i4 += gridDim.x * 256u) {
        const unsigned i = i4 * 4u;
        const unsigned row = (unsigned)conv_fdiv((int)i, (int)pitch, dv_pitch);   // merged: channel; per image: n*C + c
        const unsigned j = i - row * pitch;                                        // a multiple of four
        unsigned n = 0, r = j;
        if (merged) {
            n = (unsigned)conv_fdiv((int)j, (int)PQ, dv_PQ);
            r = j - n * PQ;
        }
        unsigned pp = (unsigned)conv_fdiv((int)r, (int)Q, dv_Q), q = r - pp * Q;
        const float *src[4];
        bool ok[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const unsigned plane = merged ? n * C + row : row;
            ok[e] = j + e < NPQ;
            src[e] = X + (size_t)plane * HW + pp * rowstep + q * sw;
            // step to the next output pixel: along the row, then to the next row, then to the next image
            ++r;
            if (++q == Q) { q = 0; ++pp; }
            if (r == PQ) { r = 0; pp = 0; q = 0; ++n; }
        }
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = ok[e] ? gather_round(__ldg(src[e])) : 0.f;
        Xg4[i4] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

// Per-image layout, Q a multiple of 4, W a multiple of 4, column stride 1 or 2: four outputs per
// thread from one or two aligned 16-byte loads, one 16-byte store.
template <int SW>
__global__ void __launch_bounds__(256)
gather1x1_vec_kernel(const float4 *__restrict__ X4, float4 *__restrict__ Xg4, unsigned total4, unsigned PQ4,
                     unsigned Q4, unsigned HW4, unsigned rowstep4) {
    tc::pdl_launch_dependents();
    for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < total4; i += gridDim.x * 256u) {
        const unsigned plane = i / PQ4, r = i - plane * PQ4;
        const unsigned p = r / Q4, q4 = r - p * Q4;
        const float4 *src = X4 + (size_t)plane * HW4 + p * rowstep4 + q4 * SW;
        float4 o;
        if (SW == 1) {
            o = __ldg(src);
        } else {
            const float4 a = __ldg(src), b = __ldg(src + 1);
            o = make_float4(a.x, a.z, b.x, b.z);
        }
        o.x = gather_round(o.x); o.y = gather_round(o.y); o.z = gather_round(o.z); o.w = gather_round(o.w);
        Xg4[i] = o;
    }
}

// Depthwise convolution with unit stride and dilation (group = C = M), the HBM-bound case: 2.25
// flop per byte, so the only thing that matters is to move each plane once with few instructions.
// A thread owns a strip of 4 output columns by ROWS output rows of one (image, channel) plane, reads
// the KH + ROWS - 1 input rows it needs straight from global memory (neighbouring threads' overlapping
// reads are served by L1) and keeps the window in registers: with ROWS = 4 and a 3x3 filter, 18 loads
// and 144 FMAs for 16 outputs, every input row fetched 1.5 times instead of twice with ROWS = 2.  VEC: the row pitch and the left pad allow one aligned 16-byte load per row for the
// strip's middle columns; otherwise every column is loaded on its own.
template <int KH, int KW, bool VEC, int ROWS>
__global__ void __launch_bounds__(256)
conv2d_depthwise_unit_kernel(const ConvGeom g, const float *__restrict__ X, const float *__restrict__ W,
                             const float *__restrict__ B, const float *__restrict__ R, float *__restrict__ Y,
                             unsigned items, unsigned Q4, unsigned P2, double inv_Q4, double inv_P2) {
    constexpr int WIN = KW + 3;                // input columns a strip of 4 outputs touches
    tc::pdl_launch_dependents();               // (launched plainly itself) lets the next kernel set up early
    const unsigned i = blockIdx.x * 256u + threadIdx.x;
    if (i >= items) return;
    // i = (plane * P2 + row group) * Q4 + column quad (P2 = row groups per plane); quotients by reciprocal multiplication in
    // double (right for 31-bit operands up to one unit, which the two comparisons repair)
    unsigned t = __double2uint_rd((double)i * inv_Q4);
    if (t * Q4 > i) --t;
    if ((t + 1) * Q4 <= i) ++t;
    const unsigned q4 = i - t * Q4;
    unsigned plane = __double2uint_rd((double)t * inv_P2);
    if (plane * P2 > t) --plane;
    if ((plane + 1) * P2 <= t) ++plane;
    const int p0 = (int)(t - plane * P2) * ROWS, q0 = (int)q4 * 4;
    const int c = (int)(plane % (unsigned)g.C);

    float w[KH * KW];
#pragma unroll
    for (int k = 0; k < KH * KW; ++k) w[k] = __ldg(W + (size_t)c * (KH * KW) + k);
    const float bias = B ? __ldg(B + c) : 0.f;
    float acc[ROWS][4];
#pragma unroll
    for (int k = 0; k < ROWS; ++k)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[k][j] = bias;

    const float *xp = X + (size_t)plane * g.H * g.W;
    const int iw0 = q0 - g.pl;
    // Every input row of the window is requested before the first FMA: the kernel is bound by the
    // latency of these loads, so each thread keeps all of them in flight at once.
    float v[KH + ROWS - 1][WIN];
#pragma unroll
    for (int rr = 0; rr < KH + ROWS - 1; ++rr) {
        const int ih = p0 - g.pt + rr;
#pragma unroll
        for (int k = 0; k < WIN; ++k) v[rr][k] = 0.f;
        if ((unsigned)ih < (unsigned)g.H) {
            const float *row = xp + (size_t)ih * g.W;
            if (VEC) {
                // pl == 1: columns q0-1 .. q0+KW+1; q0 .. q0+3 are one aligned float4
                if (iw0 >= 0) v[rr][0] = __ldg(row + iw0);
                if (q0 + 3 < g.W) {
                    const float4 m = __ldg(reinterpret_cast<const float4 *>(row + q0));
                    v[rr][1] = m.x; v[rr][2] = m.y; v[rr][3] = m.z; v[rr][4] = m.w;
                } else {
#pragma unroll
                    for (int k = 1; k < 5; ++k) if (iw0 + k < g.W) v[rr][k] = __ldg(row + iw0 + k);
                }
#pragma unroll
                for (int k = 5; k < WIN; ++k) if (iw0 + k < g.W) v[rr][k] = __ldg(row + iw0 + k);
            } else {
#pragma unroll
                for (int k = 0; k < WIN; ++k) if ((unsigned)(iw0 + k) < (unsigned)g.W) v[rr][k] = __ldg(row + iw0 + k);
            }
        }
    }
#pragma unroll
    for (int rr = 0; rr < KH + ROWS - 1; ++rr) {
        // input row rr is filter row rr - k of output row p0 + k
#pragma unroll
        for (int k = 0; k < ROWS; ++k) {
            if (rr - k >= 0 && rr - k < KH) {
#pragma unroll
                for (int s = 0; s < KW; ++s)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[k][j] = fmaf(v[rr][j + s], w[(rr - k) * KW + s], acc[k][j]);
            }
        }
    }
    float *yp = Y + ((size_t)plane * g.P + p0) * g.Q + q0;
#pragma unroll
    for (int k = 0; k < ROWS; ++k) {
        float *a = acc[k];
        if (p0 + k >= g.P) break;
        if (R) {
            const float *rr = R + (yp - Y) + (size_t)k * g.Q;
#pragma unroll
            for (int j = 0; j < 4; ++j) if (q0 + j < g.Q) a[j] += __ldg(rr + j);
        }
        if (g.relu) {
#pragma unroll
            for (int j = 0; j < 4; ++j) a[j] = a[j] > 0.f ? a[j] : 0.f;
        }
        float *yr = yp + (size_t)k * g.Q;
        if (VEC && q0 + 3 < g.Q) {
            *reinterpret_cast<float4 *>(yr) = make_float4(a[0], a[1], a[2], a[3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) if (q0 + j < g.Q) yr[j] = a[j];
        }
    }
}

template <int KH, int KW>
int launch_depthwise_unit(const ConvGeom &g, const float *X, const float *W, const float *B, const float *R, float *Y,
                          cudaStream_t st) {
    // four output rows per thread where that still gives every SM a few thousand threads, else two
    const bool rows4 = (long long)g.N * g.C * ((g.P + 3) / 4) * ((g.Q + 3) / 4) >= 148LL * 2048 * 2;
    const int rows = rows4 ? 4 : 2;
    const unsigned Q4 = (unsigned)((g.Q + 3) / 4), P2 = (unsigned)((g.P + rows - 1) / rows);
    const long long items = (long long)g.N * g.C * P2 * Q4;
    const unsigned blocks = (unsigned)((items + 255) / 256);
    // aligned 16-byte accesses: every input and output row starts on a 16-byte boundary
    const bool vec = g.pl == 1 && g.W % 4 == 0 && g.Q % 4 == 0 &&
                     (reinterpret_cast<uintptr_t>(X) & 15) == 0 && (reinterpret_cast<uintptr_t>(Y) & 15) == 0;
    auto kern = vec ? (rows4 ? conv2d_depthwise_unit_kernel<KH, KW, true, 4> : conv2d_depthwise_unit_kernel<KH, KW, true, 2>)
                    : (rows4 ? conv2d_depthwise_unit_kernel<KH, KW, false, 4> : conv2d_depthwise_unit_kernel<KH, KW, false, 2>);
    kern<<<blocks, 256, 0, st>>>(g, X, W, B, R, Y, (unsigned)items, Q4, P2, 1.0 / (double)Q4, 1.0 / (double)P2);
    count_launch();
    return (int)cudaGetLastError();
}

bool depthwise_unit_fits(const ConvGeom &g) {
    if (!(g.Cg == 1 && g.Mg == 1 && g.sh == 1 && g.sw == 1 && g.dh == 1 && g.dw == 1)) return false;
    if (!((g.kH == 3 && g.kW == 3) || (g.kH == 5 && g.kW == 5))) return false;
    const long long items = (long long)g.N * g.C * ((g.P + 1) / 2) * ((g.Q + 3) / 4);
    return items < (1LL << 31) - 256;
}

void depthwise_window(const ConvGeom &g, int &rows, int &cols, int &pitch) {
    rows = (kDwTP - 1) * g.sh + (g.kH - 1) * g.dh + 1;
    cols = (kDwTQ - 1) * g.sw + (g.kW - 1) * g.dw + 1;
    pitch = cols | 1;                          // odd pitch: strided column reads stay conflict-free
}

}  // namespace

bool simt_depthwise_supports(const ConvGeom &g) {
    if (!(g.Cg == 1 && g.Mg == 1)) return false;
    int rows, cols, pitch;
    depthwise_window(g, rows, cols, pitch);
    const long long floats = (long long)rows * pitch + (long long)g.kH * g.kW;
    if (floats * 4 > 96 * 1024) return false;
    const long long q_tiles = (g.Q + kDwTQ - 1) / kDwTQ, p_tiles = (g.P + kDwTP - 1) / kDwTP;
    return q_tiles * p_tiles * (long long)g.N * g.C <= 2147483647LL;
}

int launch_gather1x1(const ConvGeom &g, const float *X, float *Xg, long long pitch, bool merged, void *stream) {
    const long long total = merged ? (long long)g.C * pitch : (long long)g.N * g.C * pitch;
    cudaStream_t st = (cudaStream_t)stream;
    if (!merged && g.Q % 4 == 0 && g.W % 4 == 0 && (g.sw == 1 || g.sw == 2) && g.Q * g.sw <= g.W) {
        const long long total4 = total / 4;
        const unsigned blocks = (unsigned)std::min<long long>((total4 + 255) / 256, 148LL * 16);
        const unsigned PQ4 = g.P * g.Q / 4, Q4 = g.Q / 4, HW4 = g.H * g.W / 4, rowstep4 = g.sh * g.W / 4;
        if (g.sw == 1)
            gather1x1_vec_kernel<1><<<blocks, 256, 0, st>>>(reinterpret_cast<const float4 *>(X),
                                                           reinterpret_cast<float4 *>(Xg), (unsigned)total4, PQ4, Q4,
                                                           HW4, rowstep4);
        else
            gather1x1_vec_kernel<2><<<blocks, 256, 0, st>>>(reinterpret_cast<const float4 *>(X),
                                                           reinterpret_cast<float4 *>(Xg), (unsigned)total4, PQ4, Q4,
                                                           HW4, rowstep4);
    } else if (pitch % 4 == 0) {
        const long long total4 = total / 4;
        const unsigned blocks = (unsigned)std::min<long long>((total4 + 255) / 256, 148LL * 32);
        gather1x1_quad_kernel<<<blocks, 256, 0, st>>>(X, reinterpret_cast<float4 *>(Xg), (unsigned)total4, (unsigned)pitch,
                                                      (unsigned)(merged ? g.N * g.P * g.Q : g.P * g.Q),
                                                      (unsigned)(g.P * g.Q), (unsigned)g.Q, (unsigned)g.C,
                                                      (unsigned)(g.H * g.W), (unsigned)(g.sh * g.W), (unsigned)g.sw,
                                                      merged ? 1 : 0, conv_divisor((int)pitch), conv_divisor(g.P * g.Q),
                                                      conv_divisor(g.Q));
    } else {
        const unsigned blocks = (unsigned)std::min<long long>((total + 255) / 256, 148LL * 64);
        gather1x1_kernel<<<blocks, 256, 0, st>>>(X, Xg, (unsigned)total, (unsigned)pitch,
                                                 (unsigned)(merged ? g.N * g.P * g.Q : g.P * g.Q), (unsigned)(g.P * g.Q),
                                                 (unsigned)g.Q, (unsigned)g.C, (unsigned)(g.H * g.W),
                                                 (unsigned)(g.sh * g.W), (unsigned)g.sw, merged ? 1 : 0,
                                                 conv_divisor((int)pitch), conv_divisor(g.P * g.Q), conv_divisor(g.Q));
    }
    count_launch();
    return (int)cudaGetLastError();
}

int launch_simt_depthwise(const ConvGeom &g, const float *X, const float *W, const float *B, const float *R, float *Y,
                          void *stream) {
    if (depthwise_unit_fits(g)) {
        if (g.kH == 3) return launch_depthwise_unit<3, 3>(g, X, W, B, R, Y, (cudaStream_t)stream);
        return launch_depthwise_unit<5, 5>(g, X, W, B, R, Y, (cudaStream_t)stream);
    }
    int rows, cols, pitch;
    depthwise_window(g, rows, cols, pitch);
    const int q_tiles = (g.Q + kDwTQ - 1) / kDwTQ, p_tiles = (g.P + kDwTP - 1) / kDwTP;
    const size_t smem = ((size_t)rows * pitch + (size_t)g.kH * g.kW) * sizeof(float);
    if (smem > 48 * 1024) {
        const cudaError_t e =
            cudaFuncSetAttribute(conv2d_depthwise_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        if (e != cudaSuccess) return (int)e;
    }
    const unsigned blocks = (unsigned)((long long)q_tiles * p_tiles * g.N * g.C);
    conv2d_depthwise_kernel<<<blocks, kDwThreads, smem, (cudaStream_t)stream>>>(g, X, W, B, R, Y, q_tiles, p_tiles, rows,
                                                                              cols, pitch);
    count_launch();
    return (int)cudaGetLastError();
}

int launch_simt_conv(const ConvGeom &g, const float *X, const float *W, const float *B, const float *R, float *Y,
                     void *stream) {
    const long long PQ = (long long)g.P * g.Q;
    const int pixel_tiles = (int)((PQ + kDirectThreads - 1) / kDirectThreads);
    const long long gx = (long long)pixel_tiles * g.N;
    if (gx > 2147483647LL) return (int)cudaErrorInvalidConfiguration;
    const int MT = g.Mg >= 8 ? 8 : (g.Mg >= 4 ? 4 : 1);
    const int m_tiles_per_group = (g.Mg + MT - 1) / MT;
    const long long m_tiles = (long long)m_tiles_per_group * g.group;
    dim3 grid((unsigned)gx, (unsigned)(m_tiles > 65535 ? 65535 : m_tiles), 1);
    cudaStream_t st = (cudaStream_t)stream;
    if (MT == 8)
        conv2d_direct_kernel<8><<<grid, kDirectThreads, 0, st>>>(g, X, W, B, R, Y, pixel_tiles, m_tiles_per_group);
    else if (MT == 4)
        conv2d_direct_kernel<4><<<grid, kDirectThreads, 0, st>>>(g, X, W, B, R, Y, pixel_tiles, m_tiles_per_group);
    else
        conv2d_direct_kernel<1><<<grid, kDirectThreads, 0, st>>>(g, X, W, B, R, Y, pixel_tiles, m_tiles_per_group);
    count_launch();
    return (int)cudaGetLastError();
}

}  // namespace onnxb
