// Optional in-kernel instrumentation of the two tensor-core kernels.  Nothing here is compiled unless the
// library is built with -DONNXB_PROFILE (cycle accounting per warp role and an event log of CTA 0) or
// -DONNXB_CHECK (index checks in the weight-packing kernel); in a normal build every macro below is
// empty and no symbol is added.  The including file selects its part with ONNXB_DEBUG_HOOKS_CONV or
// ONNXB_DEBUG_HOOKS_GEMM.
#pragma once
#include <cuda_runtime.h>

#if defined(ONNXB_PROFILE) && defined(ONNXB_DEBUG_HOOKS_CONV)
__device__ long long g_prof[148 * 16];
#define PROF_DECL long long pt_ = clock64(), pacc_[6] = {0, 0, 0, 0, 0, 0}
#define PROF_MARK(k) do { long long n_ = clock64(); pacc_[k] += n_ - pt_; pt_ = n_; } while (0)
#define PROF_FLUSH(base) do { if (blockIdx.x < 148) for (int k_ = 0; k_ < 6; ++k_) g_prof[blockIdx.x * 16 + (base) + k_] = pacc_[k_]; } while (0)
// event log of CTA 0: kind k (0..8; 8 = phases of the kernel as a whole), sequence number i (0..63) -> clock
__device__ long long g_log[9 * 64];
#define LOG(k, i) do { if (blockIdx.x == 0 && (i) < 64) g_log[(k) * 64 + (i)] = clock64(); } while (0)
extern "C" int onnxb_dbg_profile(long long *out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_prof, sizeof(long long) * 148 * 16);
    static long long zeros[148 * 16];
    cudaMemcpyToSymbol(g_prof, zeros, sizeof zeros);
    return 0;
}
extern "C" int onnxb_dbg_log(long long *out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_log, sizeof(long long) * 9 * 64);
    return 0;
}
#else
#define LOG(k, i) do {} while (0)
#define PROF_DECL do {} while (0)
#define PROF_MARK(k) do {} while (0)
#define PROF_FLUSH(base) do {} while (0)
#endif

#if defined(ONNXB_CHECK) && defined(ONNXB_DEBUG_HOOKS_CONV)
__device__ long long g_chk[8];
#define CHK(cond, code, val) if (!(cond)) { if (atomicCAS((unsigned long long *)&g_chk[0], 0ull, (unsigned long long)(code)) == 0ull) { g_chk[1] = (long long)(val); g_chk[2] = blockIdx.x; g_chk[3] = threadIdx.x; } continue; }
extern "C" int onnxb_dbg_check(long long *out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_chk, sizeof(long long) * 8);
    return 0;
}
#else
#define CHK(cond, code, val)
#endif

#if defined(ONNXB_PROFILE) && defined(ONNXB_DEBUG_HOOKS_GEMM)
__device__ long long g_gprof[148 * 16];
#define GP_DECL long long pt_ = clock64(), pacc_[6] = {0, 0, 0, 0, 0, 0}
#define GP_MARK(k) do { long long n_ = clock64(); pacc_[k] += n_ - pt_; pt_ = n_; } while (0)
#define GP_FLUSH(base, n) do { if (blockIdx.x < 148) for (int k_ = 0; k_ < n; ++k_) g_gprof[blockIdx.x * 16 + (base) + k_] = pacc_[k_]; } while (0)
__device__ long long g_glog[4 * 128];
#define GLOG(k, i) do { if (blockIdx.x == 0 && (i) < 128) g_glog[(k) * 128 + (i)] = clock64(); } while (0)
extern "C" int onnxb_dbg_glog(long long *out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_glog, sizeof(long long) * 4 * 128);
    return 0;
}
extern "C" int onnxb_dbg_gprofile(long long *out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_gprof, sizeof(long long) * 148 * 16);
    return 0;
}
#else
#define GLOG(k, i) do {} while (0)
#define GP_DECL do {} while (0)
#define GP_MARK(k) do {} while (0)
#define GP_FLUSH(base, n) do {} while (0)
#endif
