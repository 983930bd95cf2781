/*
 * fp64 CPU oracle for ONNX Conv (2-D, NCHW) and ONNX Gemm.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product library includes, links or
 * calls this file; it shares no code with the CUDA path.
 *
 * The paper names convolution and Gemm among the operators its compiler lowers
 * (Sec. 4.1) and builds Gemm from MatMul followed by Add (Sec. 3.4.3,
 * MulAddToGemmPattern); it defers the arithmetic of both to the ONNX standard
 * (Sec. 2.1).  Because the result has a plain definition, this file is that
 * definition written out: one loop per index of the sum, evaluated in double
 * precision from the float inputs, no blocking, no reordering.
 *
 * Besides the result Y each routine returns S, the sum of the absolute values
 * of the same products, which the parity tolerance |gpu - Y| <= 1e-3*S + 1e-5
 * is built from.
 *
 * Parity unpinned: behaviour on NaN / Inf / -0 inputs (Relu of NaN is taken as
 * +0 here), and auto_pad=SAME_* combined with dilation > 1 (resolved on the
 * Python side of the oracle with the dilated kernel extent).
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int onnx_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * ONNX Conv, 2-D (operator named in Sec. 4.1; semantics per the ONNX standard,
 * Sec. 2.1):
 *
 *   Y[n,m,p,q] = B[m] + sum_{c<C/g} sum_{r<kH} sum_{s<kW}
 *                  Xpad[n, (m div (M/g))*(C/g) + c, p*sh + r*dh - pt, q*sw + s*dw - pl] * W[m,c,r,s]
 *
 * Xpad is X inside [0,H)x[0,W) and 0 outside; the kernel is not flipped.
 * P and Q are supplied by the caller (the Python shape resolver of the oracle).
 * relu != 0 applies v > 0 ? v : +0 afterwards.
 *
 * X [N,C,H,Wd]  W [M,C/g,kH,kW]  B [M] or NULL   (float, dense row-major)
 * Y,S [N,M,P,Q] (double)
 */
int onnx_oracle_conv2d(const float *X, const float *W, const float *B,
                       int64_t N, int64_t C, int64_t H, int64_t Wd,
                       int64_t M, int64_t kH, int64_t kW,
                       int64_t pt, int64_t pl,
                       int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                       int64_t group, int64_t P, int64_t Q, int relu,
                       double *Y, double *S)
{
    if (group <= 0 || C % group || M % group) return 1;
    const int64_t Cg = C / group;   /* input channels per group  */
    const int64_t Mg = M / group;   /* output channels per group */
    int64_t nm;
#pragma omp parallel for schedule(dynamic, 1)
    for (nm = 0; nm < N * M; ++nm) {
        const int64_t n = nm / M, m = nm % M;
        const int64_t g = m / Mg;
        for (int64_t p = 0; p < P; ++p) {
            for (int64_t q = 0; q < Q; ++q) {
                double acc = 0.0, mag = 0.0;
                for (int64_t c = 0; c < Cg; ++c) {
                    const int64_t cin = g * Cg + c;
                    for (int64_t r = 0; r < kH; ++r) {
                        const int64_t ih = p * sh + r * dh - pt;
                        if (ih < 0 || ih >= H) continue;          /* zero padding */
                        for (int64_t s = 0; s < kW; ++s) {
                            const int64_t iw = q * sw + s * dw - pl;
                            if (iw < 0 || iw >= Wd) continue;     /* zero padding */
                            const double x = (double)X[((n * C + cin) * H + ih) * Wd + iw];
                            const double w = (double)W[((m * Cg + c) * kH + r) * kW + s];
                            acc += x * w;
                            mag += fabs(x * w);
                        }
                    }
                }
                if (B) acc += (double)B[m];
                if (relu) acc = acc > 0.0 ? acc : 0.0;
                const int64_t o = ((n * M + m) * P + p) * Q + q;
                Y[o] = acc;
                if (S) S[o] = mag;
            }
        }
    }
    return 0;
}

/*
 * ONNX Gemm (Sec. 3.4.3: Gemm(m1, m2, m3) stands for Add(MatMul(m1, m2), m3);
 * the scaling and transposition attributes come from the ONNX standard):
 *
 *   Y[i,j] = alpha * sum_k A'[i,k] * B'[k,j] + beta * Cb[i,j]
 *
 * A' = transA ? A^T : A, B' = transB ? B^T : B.  A is stored [M,K] (or [K,M]
 * when transA), B is stored [K,N] (or [N,K] when transB).  Cb is C broadcast to
 * [M,N]: c_stride_i / c_stride_j are the element strides of C along i and j
 * (0 for a broadcast axis); C == NULL omits the term.
 * S[i,j] = |alpha| * sum_k |A'[i,k] * B'[k,j]|.
 */
int onnx_oracle_gemm(const float *A, const float *B, const float *C,
                     int64_t M, int64_t N, int64_t K,
                     int transA, int transB, double alpha, double beta,
                     int64_t c_stride_i, int64_t c_stride_j, int relu,
                     double *Y, double *S)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0, mag = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double a = (double)(transA ? A[k * M + i] : A[i * K + k]);
                const double b = (double)(transB ? B[j * K + k] : B[k * N + j]);
                acc += a * b;
                mag += fabs(a * b);
            }
            double y = alpha * acc;
            if (C) y += beta * (double)C[i * c_stride_i + j * c_stride_j];
            if (relu) y = y > 0.0 ? y : 0.0;
            Y[i * N + j] = y;
            if (S) S[i * N + j] = fabs(alpha) * mag;
        }
    }
    return 0;
}
