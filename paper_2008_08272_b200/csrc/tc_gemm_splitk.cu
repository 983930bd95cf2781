// Split-K form of the TF32 tensor-core GEMM for problems with few output tiles and a long reduction
// (ONNX Gemm with a small M: a classifier head, Sec. 3.4.3 / 4.2):
//     Y (M x N) = relu?( alpha * A' (M x K) * B' (K x N) + beta * C ),   M <= 128.
// The ordinary kernel gives such a problem one serial K loop per tile on a fraction of the SMs.  Here a
// cluster of S CTAs shares one 128 x BN output tile: CTA r of the cluster reduces K-blocks
// [r * kb_per, (r + 1) * kb_per) into its own TMEM accumulator (TMA -> shared memory -> tcgen05.mma, as in
// tc_gemm.cu), parks the partial tile in its shared memory, and after a cluster barrier every CTA sums
// one slice of the tile's rows over all S partials through distributed shared memory
// (ld.shared::cluster), applies the epilogue and stores it.  The S partials of an element are always
// added in rank order, so the result does not depend on timing.
// Operands are rounded to TF32 (nearest) inside the kernel: while a stage waits for its MMAs, the four
// epilogue warps, otherwise idle during the main loop, round it in place in shared memory, so callers pass
// A and B as they are and need no rounding pass in front (the tensor core would truncate them).
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>

#include "common.h"
#include "tc_common.cuh"
#include "tc_host.h"

namespace onnxb {

namespace {

using namespace tc;

constexpr int kBM = 128, kBK = 32;
constexpr int kThreads = 192;                 // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue + reduction
constexpr int kMaxStages = 8;
constexpr int kABytes = kBM * kBK * 4;        // 16 KB
constexpr int kPitch = kBM + 4;               // floats between the columns of the parked partial tile (132: both the
                                              // row-wise writes and the column-wise reads are conflict-free)
constexpr int kSmemLimit = 232448;

struct SkParams {
    int M, N, K;
    int b_mn;                  // B' is MN-major (B stored [K, N]); A' is always K-major here
    int BN, S, num_kb, kb_per, num_stages, rows_per;
    uint32_t stage_bytes, idesc;
    float alpha, beta;
    const float *C;
    long long c_si, c_sj;
    int relu;
    float *Y;
    long long y_ld;
    unsigned int *err;
};

__device__ __forceinline__ float ld_cluster_f32(uint32_t cluster_addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(cluster_addr) : "memory");
    return v;
}

__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_splitk_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const SkParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *stages = smem;
    float *partial = reinterpret_cast<float *>(smem + (size_t)p.num_stages * p.stage_bytes);     // [BN][kPitch]
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(partial) + (size_t)p.BN * kPitch * 4);
    uint64_t *full = bars, *empty = bars + kMaxStages, *ready = bars + 2 * kMaxStages, *acc_full = bars + 3 * kMaxStages;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(bars + 3 * kMaxStages + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const int tn = blockIdx.x / p.S;                                  // the cluster's column tile
    const int kb0 = rank * p.kb_per, kb1 = min(p.num_kb, kb0 + p.kb_per);
    const int nkb = max(kb1 - kb0, 0);                                // K-blocks this CTA reduces (0: a rank past the end)

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
            mbar_init(&ready[s], 4);               // the four rounding warps
        }
        mbar_init(acc_full, 1);
        mbar_fence_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(tmem_holder, 64);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;
    pdl_launch_dependents();
    pdl_wait();                 // everything above overlapped the previous kernel's tail

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (lane 0: A, lanes 1..: B)
        const int nb = p.b_mn ? p.BN / 32 : 1;                        // copies of B per stage
        int stage = 0;
        uint32_t phase = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
            mbar_wait(&empty[stage], phase ^ 1, p.err, 40);
            if (lane == 0) mbar_arrive_expect_tx(&full[stage], p.stage_bytes);
            __syncwarp();
            uint8_t *dst = stages + (size_t)stage * p.stage_bytes;
            if (lane == 0) {
                tma_load_2d(dst, &tmA, &full[stage], kb * kBK, 0);
            } else if (lane <= nb) {
                if (!p.b_mn) tma_load_2d(dst + kABytes, &tmB, &full[stage], kb * kBK, tn * p.BN);
                else tma_load_2d(dst + kABytes + (lane - 1) * 4096, &tmB, &full[stage], tn * p.BN + (lane - 1) * 32, kb * kBK);
            }
            if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one() && nkb > 0) {
            const uint64_t a_tmpl = make_smem_desc(0, 16, 1024, kSwizzle128B);
            const uint64_t b_tmpl = p.b_mn ? make_smem_desc(0, 4096, 512, kSwizzle128B32) : make_smem_desc(0, 16, 1024, kSwizzle128B);
            const uint32_t a_hi = (uint32_t)(a_tmpl >> 32), b_hi = (uint32_t)(b_tmpl >> 32);
            const uint32_t a_lo_c = (uint32_t)a_tmpl, b_lo_c = (uint32_t)b_tmpl;
            const uint32_t b_k16 = (p.b_mn ? 1024u : 32u) >> 4;
            int stage = 0;
            uint32_t phase = 0;
            for (int i = 0; i < nkb; ++i) {
                mbar_wait(&ready[stage], phase, p.err, 41);       // landed and rounded
                tc_fence_after_sync();
                const uint32_t sA = smem_u32(stages + (size_t)stage * p.stage_bytes);
                const uint32_t a16 = sA >> 4, b16 = (sA + kABytes) >> 4;
#pragma unroll
                for (int k = 0; k < kBK / 8; ++k)
                    mma_tf32_lohi(tmem_base, a_lo_c | ((a16 + (uint32_t)k * 2u) & 0x3FFFu), a_hi,
                                  b_lo_c | ((b16 + (uint32_t)k * b_k16) & 0x3FFFu), b_hi, p.idesc, (i | k) != 0);
                mma_commit(&empty[stage]);
                if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
            }
            mma_commit(acc_full);
        }
    } else {
        // ------------------------------------------------------------ park this CTA's partial tile: partial[col][row]
        const int q = warp & 3;                    // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        {
            // main loop: round every landed stage to TF32 in place (elementwise, so the swizzle does not matter)
            const int t = (warp - 2) * 32 + lane;
            const int n4 = (int)(p.stage_bytes >> 4);
            int stage = 0;
            uint32_t phase = 0;
            for (int i = 0; i < nkb; ++i) {
                mbar_wait(&full[stage], phase, p.err, 43);
                float4 *st4 = reinterpret_cast<float4 *>(stages + (size_t)stage * p.stage_bytes);
                for (int j = t; j < n4; j += 128) {
                    float4 v = st4[j];
                    v.x = round_tf32(v.x); v.y = round_tf32(v.y); v.z = round_tf32(v.z); v.w = round_tf32(v.w);
                    st4[j] = v;
                }
                fence_proxy_async_smem();          // generic-proxy writes, read next by the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(&ready[stage]);
                if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
            }
        }
        if (nkb > 0) {
            mbar_wait(acc_full, 0, p.err, 42);
            tc_fence_after_sync();
        }
        for (int c0 = 0; c0 < p.BN; c0 += 32) {
            uint32_t v[32];
            if (nkb > 0) {
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = 0u;
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) partial[(c0 + j) * kPitch + row] = __uint_as_float(v[j]);
        }
        tc_fence_before_sync();
    }

    // every CTA's partial tile is in its shared memory
    cluster_sync_all();

    if (warp >= 2) {
        // ------------------------------------------------------------ reduce this CTA's slice of rows over the cluster
        const int t = (warp - 2) * 32 + lane;      // 0..127
        const int row_lo = rank * p.rows_per;
        const int n_items = p.rows_per * p.BN;
        const uint32_t part_addr = smem_u32(partial);
        for (int idx = t; idx < n_items; idx += 128) {
            const int rr = idx / p.BN, col = idx - rr * p.BN;
            const int row = row_lo + rr, gcol = tn * p.BN + col;
            if (row >= p.M || gcol >= p.N) continue;
            const uint32_t off = (uint32_t)(col * kPitch + row) * 4u;
            float acc = 0.f;
            for (int s = 0; s < p.S; ++s) acc += ld_cluster_f32(map_to_cta(part_addr + off, (uint32_t)s));
            float x = p.alpha * acc;
            if (p.C) x = fmaf(p.beta, __ldg(p.C + (long long)row * p.c_si + (long long)gcol * p.c_sj), x);
            if (p.relu) x = fmaxf(x, 0.f);
            p.Y[(long long)row * p.y_ld + gcol] = x;
        }
    }

    // no CTA leaves while a peer may still read its partial tile
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 64);
    }
}

struct SkChoice {
    int BN, S;
};

// Split-K pays when the ordinary kernel would leave most SMs idle on a long reduction.
bool choose(const TcGemmProblem &g, SkChoice &c) {
    if (g.batch != 1 || g.a_mn_major || g.row_bias || g.residual || g.y_split) return false;
    if (g.M > kBM || g.K < 512 || g.N < 32) return false;
    if (g.a_ld % 4 || g.b_ld % 4) return false;
    const int num_kb = (g.K + kBK - 1) / kBK;
    int best = 0;
    for (int S : {2, 4, 8})
        for (int BN : {64, 32}) {
            const int ctas = ((g.N + BN - 1) / BN) * S;
            if (ctas > 148 || num_kb / S < 4) continue;
            if (ctas > best) { best = ctas; c.BN = BN; c.S = S; }      // at equal count the smaller split (fewer partials)
        }
    if (const char *e = getenv("ONNXB_GEMM_SPLITK")) {    // "BN,S": pin the shape for A/B measurements
        int bn = 0, sp = 0;
        if (sscanf(e, "%d,%d", &bn, &sp) == 2 && (bn == 32 || bn == 64) && (sp == 2 || sp == 4 || sp == 8) &&
            num_kb / sp >= 1) {
            c.BN = bn;
            c.S = sp;
            return true;
        }
    }
    // worth it when the ordinary kernel (128 x 32 tiles at best) would occupy a third of the SMs or fewer
    return best >= 64 && (g.N + 31) / 32 <= 48;
}

}  // namespace

bool tc_gemm_splitk_fits(const TcGemmProblem &g) {
    SkChoice c;
    if (const char *e = getenv("ONNXB_GEMM_SPLITK"))      // "0": never (for A/B measurements)
        if (e[0] == '0') return false;
    return choose(g, c);
}

int launch_tc_gemm_splitk(const TcGemmProblem &g, void *stream) {
    using namespace tc_host;
    SkChoice c;
    if (!choose(g, c)) return (int)cudaErrorInvalidValue;
    SkParams p{};
    p.M = g.M; p.N = g.N; p.K = g.K;
    p.b_mn = g.b_mn_major;
    p.BN = c.BN; p.S = c.S;
    p.num_kb = (g.K + kBK - 1) / kBK;
    p.kb_per = (p.num_kb + p.S - 1) / p.S;
    p.rows_per = (g.M + p.S - 1) / p.S;
    p.stage_bytes = (uint32_t)(kABytes + p.BN * 128);
    p.num_stages = std::min(kMaxStages, std::max(2, p.kb_per));
    p.idesc = tc::make_idesc_tf32(kBM, p.BN, 0, p.b_mn);
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = g.C; p.c_si = g.c_si; p.c_sj = g.c_sj;
    p.relu = g.relu;
    p.Y = g.Y; p.y_ld = g.y_ld;
    p.err = device_status_ptr();
    if (!p.err) return (int)cudaErrorUnknown;

    CUtensorMap tmA, tmB;
    {
        const uint64_t dims[2] = {(uint64_t)g.K, (uint64_t)g.M};
        const uint64_t str[1] = {(uint64_t)g.a_ld * 4};
        const uint32_t box[2] = {kBK, kBM};
        if (!make_tmap(&tmA, g.A, 2, dims, str, box, kTmapSwizzle128)) return (int)cudaErrorInvalidValue;
    }
    if (!p.b_mn) {
        const uint64_t dims[2] = {(uint64_t)g.K, (uint64_t)g.N};
        const uint64_t str[1] = {(uint64_t)g.b_ld * 4};
        const uint32_t box[2] = {kBK, (uint32_t)p.BN};
        if (!make_tmap(&tmB, g.B, 2, dims, str, box, kTmapSwizzle128)) return (int)cudaErrorInvalidValue;
    } else {
        const uint64_t dims[2] = {(uint64_t)g.N, (uint64_t)g.K};
        const uint64_t str[1] = {(uint64_t)g.b_ld * 4};
        const uint32_t box[2] = {32, kBK};
        if (!make_tmap(&tmB, g.B, 2, dims, str, box, kTmapSwizzle128Atom32)) return (int)cudaErrorInvalidValue;
    }
    const size_t smem = 1024 + (size_t)p.num_stages * p.stage_bytes + (size_t)p.BN * kPitch * 4 + 512;
    if (smem > (size_t)kSmemLimit) return (int)cudaErrorInvalidConfiguration;
    const cudaError_t ae = cudaFuncSetAttribute(tc_gemm_splitk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (ae != cudaSuccess) return (int)ae;
    const int grid = ((g.N + p.BN - 1) / p.BN) * p.S;
    const cudaError_t le = launch_pdl_cluster(tc_gemm_splitk_kernel, (unsigned)p.S, dim3(grid), dim3(kThreads), smem,
                                              (cudaStream_t)stream, tmA, tmB, p);
    count_launch();
    return (int)le;
}

}  // namespace onnxb
