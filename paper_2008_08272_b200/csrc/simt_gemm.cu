// SIMT (fp32 FMA) Gemm: Y = relu?(alpha * A' * B' + beta * Cb), ONNX Gemm
// (Sec. 3.4.3).  Used for problems too small or too oddly aligned for the
// tensor-core pipeline; accepts every transA/transB/broadcast combination.
#include <cuda_runtime.h>

#include "common.h"

namespace onnxb {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;   // block tile; 256 threads, 4x4 outputs each

__global__ void __launch_bounds__(256)
gemm_simt_kernel(const GemmProblem p, const float *__restrict__ A, const float *__restrict__ B,
                 const float *__restrict__ C, float *__restrict__ Y, int tiles_n) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];

    const int tile_m = blockIdx.x / tiles_n, tile_n = blockIdx.x % tiles_n;
    const int i0 = tile_m * BM, j0 = tile_n * BN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

    // element strides of A' (i,k) and B' (k,j) in their stored arrays
    const long long a_si = p.transA ? 1 : p.K, a_sk = p.transA ? p.M : 1;
    const long long b_sk = p.transB ? 1 : p.N, b_sj = p.transB ? p.K : 1;

    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    for (int k0 = 0; k0 < p.K; k0 += BK) {
        // 1024 elements per operand tile, 4 per thread; the fast index follows
        // whichever axis is contiguous in memory
        for (int e = threadIdx.x; e < BM * BK; e += 256) {
            int ii, kk;
            if (p.transA) { ii = e % BM; kk = e / BM; } else { kk = e % BK; ii = e / BK; }
            const int i = i0 + ii, k = k0 + kk;
            As[kk][ii] = (i < p.M && k < p.K) ? __ldg(A + i * a_si + k * a_sk) : 0.f;
        }
        for (int e = threadIdx.x; e < BN * BK; e += 256) {
            int jj, kk;
            if (p.transB) { kk = e % BK; jj = e / BK; } else { jj = e % BN; kk = e / BN; }
            const int j = j0 + jj, k = k0 + kk;
            Bs[kk][jj] = (j < p.N && k < p.K) ? __ldg(B + k * b_sk + j * b_sj) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[4], bv[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) av[a] = As[kk][ty * 4 + a];
#pragma unroll
            for (int b = 0; b < 4; ++b) bv[b] = Bs[kk][tx * 4 + b];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int i = i0 + ty * 4 + a;
        if (i >= p.M) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int j = j0 + tx * 4 + b;
            if (j >= p.N) continue;
            float v = p.alpha * acc[a][b];
            if (C) v = fmaf(p.beta, __ldg(C + i * p.c_stride_i + j * p.c_stride_j), v);
            if (p.relu) v = v > 0.f ? v : 0.f;
            Y[(size_t)i * p.N + j] = v;
        }
    }
}

}  // namespace

int launch_simt_gemm(const GemmProblem &p, const float *A, const float *B, const float *C, float *Y,
                     void *stream) {
    const long long tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    if (tiles_m * tiles_n > 2147483647LL) return (int)cudaErrorInvalidConfiguration;
    gemm_simt_kernel<<<(unsigned)(tiles_m * tiles_n), 256, 0, (cudaStream_t)stream>>>(p, A, B, C, Y, (int)tiles_n);
    count_launch();
    return (int)cudaGetLastError();
}

}  // namespace onnxb
