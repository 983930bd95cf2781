// Batched TF32 GEMM on the 5th-generation tensor cores:
//     D[b] (M x N) = A'[b] (M x K) * B'[b] (K x N),   then a fused epilogue.
//
// It serves ONNX Gemm (Sec. 3.4.3) and every 1x1, stride-1 convolution (Sec. 4.1),
// which in NCHW is one GEMM per image: Y[n] (Cout x HW) = W (Cout x C) * X[n] (C x HW).
//
// Pipeline (one persistent CTA per SM, 320 threads):
//   warp 0    TMA producer: fp32 operand tiles, 128-byte swizzled, into a ring of
//             shared-memory stages, completion signalled on mbarriers; the boxes of a
//             stage are issued by as many lanes at once;
//   warp 1    one thread issues tcgen05.mma kind::tf32 (128 x BN x 8 per instruction) into
//             one of two TMEM accumulators and commits stage releases to mbarriers;
//   warps 2-9 epilogue: tcgen05.ld the finished accumulator (while the MMA warp fills the
//             other one), apply alpha / beta*C / bias / Relu, stage 32x32 blocks in swizzled
//             shared memory and write them with TMA stores (plain stores when Y cannot be
//             described by a tensor map).  Two warps share each TMEM lane quarter and split
//             its columns, so that a scheduler has a second warp to run while one waits.
// Either operand may be K-major (reduction index contiguous) or MN-major (row/column
// index contiguous, e.g. the pixels of an NCHW image); no transposed copy is ever made.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdlib>
#include <mutex>

#include "common.h"
#define ONNXB_DEBUG_HOOKS_GEMM
#include "debug_hooks.cuh"
#include "tc_common.cuh"
#include "tc_host.h"

namespace onnxb {

namespace {

using namespace tc;

constexpr int kBM = 128;            // UMMA M: rows of D per tile (TMEM lanes)
constexpr int kBK = 32;             // fp32 elements per stage along K (one 128-byte swizzle row)
constexpr int kMaxBN = 256;         // UMMA N limit
constexpr int kMaxStages = 8;
constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr int kABytes = kBM * kBK * 4;             // 16 KB
constexpr int kStoreBufBytes = 32 * 32 * 4;        // one 32x32 fp32 block
constexpr int kStagingBytes = kEpiWarps * kStoreBufBytes;   // one block per epilogue warp
constexpr int kBarrierBytes = 512;
constexpr int kResidualBufs = 2;                    // most blocks of the residual addend in flight per epilogue warp
constexpr int kSmemLimit = 232448;                 // 227 KB opt-in maximum per CTA

struct Params {
    int M, N, K, batch;
    int a_mn, b_mn;            // operand is MN-major (else K-major)
    int a_batched, b_batched;
    int BN, tiles_m, tiles_n, num_kb, num_stages;
    uint32_t idesc, stage_bytes, tx_bytes;
    // The last tile along N is only as wide as the columns left, rounded up to 16: its MMAs take the
    // descriptor below, and each CTA of a pair stages half of THAT width (so the odd CTA's first column
    // need not be a multiple of 32, and an MN-major B is then fetched block by block).
    int nt_tail;               // width of the last tile along N
    uint32_t idesc_tail;
    float alpha, beta;
    const float *C;            // optional addend, element strides below (0 = broadcast)
    long long c_si, c_sj, c_sb;
    const float *row_bias;     // optional per-row addend (convolution bias)
    const float *R;            // optional addend laid out exactly like Y (a residual connection), added before Relu
    int r_tma;                 // R is fetched by TMA (when Y is stored by TMA: same geometry), r_bufs blocks ahead
    int r_bufs;                // 1 or 2 blocks of R in flight per epilogue warp
    uint32_t staging_bytes;    // Y staging blocks, plus the R blocks when r_tma
    int relu;
    // MN-major B in one copy per stage: a 4-D view (32 columns of a block, K row, block of 32 columns,
    // batch) lets a single box carry all of a tile's 32-column blocks in the order the MMA wants them.
    int b_big;                 // that view is in use
    int b_nblk_full;           // full 32-column blocks in a row of B (tiles reaching past them load block by block)
    // CTA pairs: two CTAs of a cluster share a 256-row tile; each loads its 128 rows of A and half of
    // the tile's B columns, the even CTA issues cta_group::2 MMAs (M = 256)
    int ctas, BNH;             // CTAs per tile; B columns staged per CTA = BN / ctas
    float *Y;                  // used by the plain-store epilogue
    long long y_ld, y_sb;
    int y_split;               // > 0: columns are groups of y_split, y_group elements apart (plain stores only)
    long long y_group;
    int y_tma;
    unsigned int *err;
};

template <int kCtas>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmBb, const __grid_constant__ CUtensorMap tmY,
               const __grid_constant__ CUtensorMap tmR, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment by pointer arithmetic on the shared array itself, so that the compiler
    // keeps treating everything derived from it as shared memory (LDS/STS, not generic accesses)
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *stages = smem;
    uint8_t *staging = smem + (size_t)p.num_stages * p.stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + p.staging_bytes);
    uint64_t *full = bars, *empty = bars + kMaxStages;
    uint64_t *tmem_full = bars + 2 * kMaxStages, *tmem_empty = tmem_full + 2;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(tmem_empty + 2);
    uint64_t *r_full = bars + 24;              // [epilogue warp][kResidualBufs]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.tiles_m * p.tiles_n * p.batch;
    const int rank = kCtas == 2 ? (int)cluster_ctarank() : 0;
    const int first_tile = blockIdx.x / kCtas, tile_step = gridDim.x / kCtas;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) {
            // issuing CTA of a pair: its own producer plus the peer's "landed" message
            mbar_init(&full[s], (kCtas == 2 && rank == 0) ? 2 : 1);
            mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&tmem_full[a], 1);
            mbar_init(&tmem_empty[a], kEpiWarps * kCtas);
        }
        for (int a = 0; a < kEpiWarps * kResidualBufs; ++a) mbar_init(&r_full[a], 1);
        mbar_fence_init();
        if (p.r_tma) prefetch_tmap(&tmR);
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (p.b_big) prefetch_tmap(&tmBb);
        if (p.y_tma) prefetch_tmap(&tmY);
    }
    if (warp == 1) {
        tmem_alloc(tmem_holder, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;
    if (kCtas == 2) cluster_sync_all();     // the peer's barriers exist before anything arrives on them
    pdl_launch_dependents();
    // Everything above overlapped the previous kernel's tail, and so does each role's own set-up below: the
    // warps that touch global memory (the producer, the epilogue warps) wait for the previous kernel just
    // before their first access; the MMA warp only ever sees what the producer hands it.

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // The TMA unit spends 70-90 cycles on every copy instruction however small it is, so a stage is
        // fetched with as few instructions as possible (an MN-major B of up to eight 4 KB blocks through
        // one 4-D box), and the whole warp runs the loop so that the copies of a stage are issued by as
        // many lanes at once instead of one thread paying its instruction latency for each.  Measured
        // on the issuing lane: 580 cycles per stage with A and B as two different copy instructions,
        // 452 with both as one instruction executed by two lanes.
        {
            int stage = 0;
            uint32_t phase = 0;
            const int na = p.a_mn ? kBM / 32 : 1;
            const int hb = p.BNH / 32;                 // 32-column blocks of B this CTA stages (MN-major B)
            // lanes [0, na): A pieces; lane na: B in one copy; lanes [na + 1, na + 1 + hb): B block by block
            const bool is_a = lane < na;
            const int jb = lane - na - 1;
            int glog_i = 0;
            (void)glog_i;
            for (int t = first_tile; t < total_tiles; t += tile_step) {
                const int tm = t % p.tiles_m;
                const int tn = (t / p.tiles_m) % p.tiles_n;
                const int b = t / (p.tiles_m * p.tiles_n);
                const int ab = p.a_batched ? b : 0, bb = p.b_batched ? b : 0;
                const int row_a = tm * kBM * kCtas + rank * kBM;        // first A row of this CTA
                const int bnh_t = (tn == p.tiles_n - 1 ? p.nt_tail : p.BN) / kCtas;     // columns this CTA stages
                const int col_b = tn * p.BN + rank * bnh_t;             // first B column of this CTA
                // do all of this CTA's blocks lie among the full ones?  Then one 4-D box brings them.
                const bool one_box = p.b_mn && p.b_big && (col_b & 31) == 0 && col_b / 32 + hb <= p.b_nblk_full;
                // block by block: only the blocks the tile needs and that hold columns of B
                // (never negative: a CTA whose first column lies past N fetches no block at all, and what it
                // expects on the stage's barrier is exactly what it issues)
                const int hb_t = col_b < p.N ? min((bnh_t + 31) / 32, (p.N - col_b + 31) / 32) : 0;
                const uint32_t tx_bytes = (p.b_mn && !one_box) ? (uint32_t)(kABytes + hb_t * 4096) : p.tx_bytes;
                // This lane's copy.  Every view has four dimensions (the plain ones end in a unit
                // dimension), so the copies of a stage are ONE instruction executed by several lanes
                // with their own coordinates; two different copy instructions would run one after the
                // other and each holds the warp for about 290 cycles.
                int c0 = 0, c1 = 0, c2 = 0, c3 = 0, d0 = 0, d1 = 0;
                bool active = false;
                uint32_t dst_off = 0;
                const CUtensorMap *tmap = &tmA;
                if (is_a) {
                    active = true;
                    dst_off = (uint32_t)lane * 4096u;
                    c2 = ab;
                    if (!p.a_mn) { c1 = row_a; d0 = kBK; }
                    else { c0 = row_a + lane * 32; d1 = kBK; }
                } else if (lane == na) {
                    tmap = &tmB;
                    dst_off = kABytes;
                    c2 = bb;
                    if (!p.b_mn) { active = true; c1 = col_b; d0 = kBK; }
                    else if (one_box) { active = true; tmap = &tmBb; c2 = col_b / 32; c3 = bb; d1 = kBK; }
                } else if (p.b_mn && !one_box && jb >= 0 && jb < hb_t) {
                    active = true;
                    tmap = &tmB;
                    dst_off = (uint32_t)kABytes + (uint32_t)jb * 4096u;
                    c0 = col_b + jb * 32;
                    c2 = bb;
                    d1 = kBK;
                }
                if (t == first_tile) pdl_wait();
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    mbar_wait(&empty[stage], phase ^ 1, p.err, 1);
                    if (lane == 0) GLOG(0, glog_i++);
                    if (lane == 0) mbar_arrive_expect_tx(&full[stage], tx_bytes);
                    __syncwarp();
                    uint8_t *dst = stages + (size_t)stage * p.stage_bytes + dst_off;
                    if (active) tma_load_4d(dst, tmap, &full[stage], c0, c1, c2, c3);
                    c0 += d0;
                    c1 += d1;
                    if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (kCtas == 2 && rank != 0) {
            // Odd CTA of a pair: the even CTA issues the MMAs; tell it when each of this CTA's stages
            // has landed (stage releases and finished accumulators come back by multicast commit).
            if (elect_one()) {
                const uint32_t peer_full = map_to_cta(smem_u32(&full[0]), 0);
                int stage = 0;
                uint32_t phase = 0;
                for (int t = first_tile; t < total_tiles; t += tile_step) {
                    for (int kb = 0; kb < p.num_kb; ++kb) {
                        mbar_wait(&full[stage], phase, p.err, 5);
                        mbar_arrive_remote(peer_full + (uint32_t)stage * 8u);
                        if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
                    }
                }
            }
        } else if (elect_one()) {
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            // Descriptor words that do not change: everything but the 14-bit start address.
            // K-major: 32 bytes further along the swizzled 128-byte rows per instruction (8-row groups
            // 1024 bytes apart).  MN-major 32-bit operands use the 128-byte swizzle with 32-byte atoms:
            // atoms of four 128-byte K rows (512 bytes apart along K), blocks of 32 rows/columns 4096
            // bytes apart; one instruction consumes eight K rows (1024 bytes).
            const uint64_t a_tmpl = p.a_mn ? make_smem_desc(0, 4096, 512, kSwizzle128B32) : make_smem_desc(0, 16, 1024, kSwizzle128B);
            const uint64_t b_tmpl = p.b_mn ? make_smem_desc(0, 4096, 512, kSwizzle128B32) : make_smem_desc(0, 16, 1024, kSwizzle128B);
            const uint32_t a_hi = (uint32_t)(a_tmpl >> 32), b_hi = (uint32_t)(b_tmpl >> 32);
            const uint32_t a_lo_c = (uint32_t)a_tmpl, b_lo_c = (uint32_t)b_tmpl;
            const uint32_t a_k16 = (p.a_mn ? 1024u : 32u) >> 4, b_k16 = (p.b_mn ? 1024u : 32u) >> 4;
            int glog_i = 0, glog_t = 0;
            (void)glog_i; (void)glog_t;
            GP_DECL;
            for (int t = first_tile; t < total_tiles; t += tile_step) {
                if (kCtas == 2) mbar_wait_cluster(&tmem_empty[acc], acc_phase ^ 1, p.err, 2);
                else mbar_wait(&tmem_empty[acc], acc_phase ^ 1, p.err, 2);
                tc_fence_after_sync();
                GP_MARK(0);
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * kMaxBN;
                const uint32_t idesc = ((t / p.tiles_m) % p.tiles_n == p.tiles_n - 1) ? p.idesc_tail : p.idesc;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (kCtas == 2) mbar_wait_cluster(&full[stage], phase, p.err, 3);
                    else mbar_wait(&full[stage], phase, p.err, 3);
                    tc_fence_after_sync();
                    GP_MARK(1);
                    GLOG(1, glog_i++);
                    const uint32_t sA = smem_u32(stages + (size_t)stage * p.stage_bytes);
                    const uint32_t a16 = sA >> 4, b16 = (sA + kABytes) >> 4;
                    const int k_left = p.K - kb * kBK;
                    const int k8 = k_left >= kBK ? kBK / 8 : (k_left + 7) / 8;
                    // one thread issues everything: keep the per-instruction work to two adds
#pragma unroll
                    for (int k = 0; k < kBK / 8; ++k) {
                        if (k < k8) {
                            if (kCtas == 2)
                                mma_tf32_lohi_pair(d_tmem, a_lo_c | ((a16 + (uint32_t)k * a_k16) & 0x3FFFu), a_hi,
                                                   b_lo_c | ((b16 + (uint32_t)k * b_k16) & 0x3FFFu), b_hi, idesc, (kb | k) != 0);
                            else
                                mma_tf32_lohi(d_tmem, a_lo_c | ((a16 + (uint32_t)k * a_k16) & 0x3FFFu), a_hi,
                                              b_lo_c | ((b16 + (uint32_t)k * b_k16) & 0x3FFFu), b_hi, idesc, (kb | k) != 0);
                        }
                    }
                    if (kCtas == 2) mma_commit_pair(&empty[stage]);
                    else mma_commit(&empty[stage]);
                    if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
                    GP_MARK(2);
                }
                if (kCtas == 2) mma_commit_pair(&tmem_full[acc]);
                else mma_commit(&tmem_full[acc]);
                GLOG(2, glog_t++);
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1;
            }
            GP_FLUSH(0, 3);
        }
    } else {
        // ------------------------------------------------------------ epilogue
        pdl_wait();
        const int q = warp & 3;                    // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;          // which half of the tile's 32-column blocks
        uint8_t *buf = staging + (warp - 2) * kStoreBufBytes;
        // residual blocks fetched by TMA, kResidualBufs in flight per warp (used when p.r_tma)
        uint8_t *rbuf = staging + kStagingBytes + (warp - 2) * p.r_bufs * kStoreBufBytes;
        uint64_t *rbar = r_full + (warp - 2) * kResidualBufs;
        const uint32_t r_mask = (uint32_t)p.r_bufs - 1, r_shift = (uint32_t)p.r_bufs - 1;
        uint32_t r_issued = 0, r_used = 0;         // blocks requested / consumed so far by this warp
        int acc = 0;
        uint32_t acc_phase = 0;
        GP_DECL;
        const uint32_t peer_tmem_empty = kCtas == 2 ? map_to_cta(smem_u32(&tmem_empty[0]), 0) : 0u;
        for (int t = first_tile; t < total_tiles; t += tile_step) {
            const int tm = t % p.tiles_m;
            const int tn = (t / p.tiles_m) % p.tiles_n;
            const int b = t / (p.tiles_m * p.tiles_n);
            const int row0 = tm * kBM * kCtas + rank * kBM + q * 32;
            const int row = row0 + lane;
            const int nchunk_all = min(p.BN / 32, (p.N - tn * p.BN + 31) / 32);
            const int c_lo = half ? (nchunk_all + 1) / 2 : 0, c_hi = half ? nchunk_all : (nchunk_all + 1) / 2;
            // request block `chunk` of R into the next slot of the warp's ring (lane 0; the slot's last
            // reader finished before the __syncwarp that precedes every call)
            auto request_r = [&](int chunk) {
                if (lane == 0) {
                    const uint32_t slot = r_issued & r_mask;
                    mbar_arrive_expect_tx(&rbar[slot], kStoreBufBytes);
                    tma_load_3d(rbuf + slot * kStoreBufBytes, &tmR, &rbar[slot], tn * p.BN + chunk * 32, row0, b);
                }
                ++r_issued;
            };
            if (p.r_tma && row0 < p.M) {
                // the tile's first blocks of R travel while the accumulator is still being computed
                for (int c = c_lo; c < c_hi && c < c_lo + p.r_bufs; ++c) request_r(c);
            }
            mbar_wait(&tmem_full[acc], acc_phase, p.err, 4);
            tc_fence_after_sync();
            GP_MARK(0);
            if (row0 < p.M) {
                const float rb = (p.row_bias && row < p.M) ? __ldg(p.row_bias + row) : 0.f;
                const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kMaxBN);
                // one 32x32 block: scale, add, activate, hand to the store path
                auto finish = [&](const uint32_t (&v)[32], int chunk) {
                    const int col0 = tn * p.BN + chunk * 32;
                    float f[32];
                    if (p.C == nullptr && p.R == nullptr) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float x = fmaf(p.alpha, __uint_as_float(v[j]), rb);
                            f[j] = p.relu ? fmaxf(x, 0.f) : x;
                        }
                    } else if (p.C == nullptr && p.r_tma) {
                        // Residual addend by TMA: the block of R lands in the warp's ring with the same 128-byte
                        // swizzle as the Y staging block, so a lane reads its row back in eight 16-byte pieces;
                        // the slot is then refilled with the block two ahead.
                        const uint32_t slot = r_used & r_mask;
                        mbar_wait(&rbar[slot], (r_used >> r_shift) & 1u, p.err, 6);
                        ++r_used;
                        const uint8_t *rb_ = rbuf + slot * kStoreBufBytes;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const float4 t4 = *reinterpret_cast<const float4 *>(rb_ + lane * 128 + ((c ^ (lane & 7)) << 4));
                            f[4 * c] = fmaf(p.alpha, __uint_as_float(v[4 * c]), rb) + t4.x;
                            f[4 * c + 1] = fmaf(p.alpha, __uint_as_float(v[4 * c + 1]), rb) + t4.y;
                            f[4 * c + 2] = fmaf(p.alpha, __uint_as_float(v[4 * c + 2]), rb) + t4.z;
                            f[4 * c + 3] = fmaf(p.alpha, __uint_as_float(v[4 * c + 3]), rb) + t4.w;
                        }
                        __syncwarp();                                             // every lane has read its row
                        if (chunk + p.r_bufs < c_hi) request_r(chunk + p.r_bufs);
                        if (p.relu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.f);
                        }
                    } else if (p.C == nullptr) {
                        // Residual addend R, laid out like Y.  A lane owns a ROW of the block, but rows are
                        // far apart in memory, so the block is fetched the other way round: lane = column,
                        // one coalesced 128-byte read per row, parked in the warp's staging buffer (same
                        // swizzle as the Y block that follows it there) and read back a row per lane.
#pragma unroll
                        for (int j = 0; j < 32; ++j) f[j] = fmaf(p.alpha, __uint_as_float(v[j]), rb);
                        if (p.y_tma && lane == 0) tma_store_wait_read<0>();      // the buffer's last Y block has gone
                        __syncwarp();
                        {
                            const int col = col0 + lane;
                            long long coff = col;
                            if (p.y_split > 0) {
                                const int grp = col / p.y_split;
                                coff = (long long)grp * p.y_group + (col - grp * p.y_split);
                            }
                            const float *rp = p.R + b * p.y_sb + (long long)row0 * p.y_ld + coff;
                            const int rows = min(32, p.M - row0);
                            float t[32];
#pragma unroll
                            for (int r = 0; r < 32; ++r) {
                                t[r] = (r < rows && col < p.N) ? __ldg(rp) : 0.f;
                                rp += p.y_ld;
                            }
#pragma unroll
                            for (int r = 0; r < 32; ++r)
                                *reinterpret_cast<float *>(buf + r * 128 + ((((lane >> 2) ^ (r & 7)) << 4) | ((lane & 3) << 2))) = t[r];
                        }
                        __syncwarp();
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const float4 t4 = *reinterpret_cast<const float4 *>(buf + lane * 128 + ((c ^ (lane & 7)) << 4));
                            f[4 * c] += t4.x; f[4 * c + 1] += t4.y; f[4 * c + 2] += t4.z; f[4 * c + 3] += t4.w;
                        }
                        if (p.relu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.f);
                        }
                        __syncwarp();                                             // every lane has read its row back
                    } else {
                        // C broadcast: walk one pointer along the row instead of forming 64-bit
                        // products per element (this branch must stay out of the C-less path)
                        const float *cp = p.C + b * p.c_sb + (long long)row * p.c_si + (long long)col0 * p.c_sj;
                        const bool row_ok = row < p.M;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            float x = fmaf(p.alpha, __uint_as_float(v[j]), rb);
                            if (row_ok && col0 + j < p.N) x = fmaf(p.beta, __ldg(cp), x);
                            cp += p.c_sj;
                            f[j] = p.relu ? fmaxf(x, 0.f) : x;
                        }
                    }
                    GP_MARK(2);
                    // Stage the 32x32 block in shared memory, row `lane`, 16-byte chunk c at position
                    // c ^ (lane % 8) (the 128-byte swizzle, conflict-free for these 16-byte stores).
                    if (p.y_tma) {
                        if (lane == 0) tma_store_wait_read<0>();   // the store that last read this buffer is done
                    }
                    __syncwarp();
                    GP_MARK(3);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4 val = make_float4(f[4 * c], f[4 * c + 1], f[4 * c + 2], f[4 * c + 3]);
                        *reinterpret_cast<float4 *>(buf + lane * 128 + ((c ^ (lane & 7)) << 4)) = val;
                    }
                    if (p.y_tma) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        GP_MARK(4);
                        if (lane == 0) {
                            tma_store_3d(&tmY, buf, col0, row0, b);
                            tma_store_commit();
                        }
                        GP_MARK(5);
                    } else {
                        // Y rows cannot be described to TMA (row pitch not a multiple of 16 bytes): read the
                        // block back transposed, lanes along the columns, and store row by row (coalesced).
                        __syncwarp();
                        const int col = col0 + lane;
                        const int rows = min(32, p.M - row0);
                        long long coff = col;
                        if (p.y_split > 0) {
                            const int grp = col / p.y_split;
                            coff = (long long)grp * p.y_group + (col - grp * p.y_split);
                        }
                        float *yp = p.Y + b * p.y_sb + (long long)row0 * p.y_ld + coff;
                        for (int r = 0; r < rows; ++r) {
                            const float val = *reinterpret_cast<const float *>(
                                buf + r * 128 + ((((lane >> 2) ^ (r & 7)) << 4) | ((lane & 3) << 2)));
                            if (col < p.N) *yp = val;
                            yp += p.y_ld;
                        }
                        __syncwarp();
                    }
                };
                // TMEM reads are software-pipelined: the next block's load is in flight while
                // the current one is finished and stored
                uint32_t va[32], vb[32];
                if (c_lo < c_hi) tmem_ld_32x32(tbase + (uint32_t)(c_lo * 32), va);
                for (int chunk = c_lo; chunk < c_hi; chunk += 2) {
                    tmem_ld_wait();
                    if (chunk + 1 < c_hi) tmem_ld_32x32(tbase + (uint32_t)((chunk + 1) * 32), vb);
                    GP_MARK(1);
                    finish(va, chunk);
                    if (chunk + 1 < c_hi) {
                        tmem_ld_wait();
                        if (chunk + 2 < c_hi) tmem_ld_32x32(tbase + (uint32_t)((chunk + 2) * 32), va);
                        GP_MARK(1);
                        finish(vb, chunk + 1);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kCtas == 2) mbar_arrive_remote(peer_tmem_empty + (uint32_t)acc * 8u);
                else mbar_arrive(&tmem_empty[acc]);
            }
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1;
        }
        if (lane == 0) tma_store_wait_all<0>();
        if (warp == 2 && lane == 0) GP_FLUSH(4, 6);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (kCtas == 2) cluster_sync_all();     // no CTA leaves while its peer may still signal it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

int pick_bn(long long tiles_m, long long n, long long batch, int num_sms, int ctas) {
    if (n <= 32 * ctas) return 32 * ctas;
    int best = 32 * ctas;
    double best_cost = 1e300;
    for (int bn = 32 * ctas; bn <= kMaxBN; bn += 32 * ctas) {
        const long long tiles = tiles_m * ((n + bn - 1) / bn) * batch;
        const long long waves = (tiles + num_sms - 1) / num_sms;
        const double cost = (double)waves * (bn + 48);
        if (cost < best_cost - 1e-9 || (cost < best_cost + 1e-9 && bn > best)) {
            best_cost = cost;
            best = bn;
        }
    }
    return best;
}

}  // namespace

// ------------------------------------------------------------------ host side
namespace tc_host {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

bool make_tmap(CUtensorMap *out, const void *base, int rank, const uint64_t *dims, const uint64_t *strides_bytes,
               const uint32_t *box, int swizzle) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bdim[5], estr[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estr[i] = 1;
        if (i > 0) gstr[i - 1] = strides_bytes[i - 1];
    }
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<void *>(base), gdim, gstr, bdim, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle == kTmapSwizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B
              : swizzle == kTmapSwizzle128Atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B
                                                 : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int num_sms() {
    static std::atomic<int> cached{0};
    int n = cached.load(std::memory_order_acquire);
    if (n == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) {
            n = v;
            cached.store(n, std::memory_order_release);
        } else {
            return 148;
        }
    }
    return n;
}

}  // namespace tc_host

bool tc_gemm_supports(const TcGemmProblem &g) {
    if (g.M < 1 || g.N < 1 || g.K < 1 || g.batch < 1) return false;
    // tensor-map strides must be multiples of 16 bytes
    if (g.a_ld % 4 || g.b_ld % 4) return false;
    if (g.batch > 1 && ((g.a_batched && g.a_bs % 4) || (g.b_batched && g.b_bs % 4))) return false;
    if ((long long)((g.M + kBM - 1) / kBM) * g.batch > 0x7fffffffLL / 4096) return false;
    return true;
}

// How many CTA pairs (clusters of two) of the pair kernel the device runs at once; queried once.
static int gemm_max_pairs() {
    static std::atomic<int> cached{-1};
    int n = cached.load(std::memory_order_acquire);
    if (n >= 0) return n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * 148);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemLimit;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc_gemm_kernel<2>, &cfg) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = tc_host::num_sms() / 2;
    }
    cached.store(n, std::memory_order_release);
    return n;
}

int launch_tc_gemm(const TcGemmProblem &g, void *stream) {
    using namespace tc_host;
    if (tc_gemm_splitk_fits(g)) return launch_tc_gemm_splitk(g, stream);      // few tiles, long reduction
    Params p{};
    p.M = g.M; p.N = g.N; p.K = g.K; p.batch = g.batch;
    p.a_mn = g.a_mn_major; p.b_mn = g.b_mn_major;
    p.a_batched = g.a_batched && g.batch > 1; p.b_batched = g.b_batched && g.batch > 1;
    const int sms = num_sms();
    // CTA pairs when the rows fill 256-row tiles: each CTA then fetches half of B.  That is what the
    // layers bound by the L2 -> shared-memory stream (small images, many channels) need: measured 7-15 %
    // faster on the 14x14 and strided 1x1 layers of ResNet-50, neutral on the HBM-bound ones.
    p.ctas = 1;
    {
        const char *e = getenv("ONNXB_GEMM_PAIR");          // "0"/"1": pin the choice for A/B measurements
        bool pair = g.M >= 256 && (g.M % 256 == 0 || g.M % 256 > 128) && g.N >= 64;
        if (e && (e[0] == '0' || e[0] == '1')) pair = e[0] == '1' && g.M > 128 && g.N >= 64;
        if (pair) p.ctas = 2;
    }
    const int units = p.ctas == 2 ? gemm_max_pairs() : sms;
    p.tiles_m = (g.M + kBM * p.ctas - 1) / (kBM * p.ctas);
    p.BN = pick_bn(p.tiles_m, g.N, g.batch, units, p.ctas);
    if (const char *e = getenv("ONNXB_GEMM_BN")) {          // pins the tile width for A/B measurements
        const int v = atoi(e);
        if (v >= 32 * p.ctas && v <= kMaxBN && v % (32 * p.ctas) == 0) p.BN = v;
    }
    p.BNH = p.BN / p.ctas;
    p.tiles_n = (g.N + p.BN - 1) / p.BN;
    p.num_kb = (g.K + kBK - 1) / kBK;
    p.stage_bytes = (uint32_t)(kABytes + p.BNH * 128);
    p.tx_bytes = p.stage_bytes;
    p.y_tma = g.y_split == 0 && (g.y_ld % 4 == 0) && (g.batch == 1 || g.y_bs % 4 == 0);
    p.R = g.C ? nullptr : g.residual;
    p.r_tma = p.R != nullptr && p.y_tma;
    // two blocks of R per epilogue warp when the operand ring keeps at least three stages beside them
    p.r_bufs = kResidualBufs;
    if ((kSmemLimit - 1024 - kBarrierBytes - kStagingBytes * (1 + kResidualBufs)) / (int)p.stage_bytes < 3) p.r_bufs = 1;
    p.staging_bytes = (uint32_t)(kStagingBytes * (p.r_tma ? 1 + p.r_bufs : 1));
    int stages = (kSmemLimit - 1024 - kBarrierBytes - (int)p.staging_bytes) / (int)p.stage_bytes;
    p.num_stages = stages > kMaxStages ? kMaxStages : stages;
    p.idesc = tc::make_idesc_tf32(kBM * p.ctas, p.BN, p.a_mn, p.b_mn);
    {
        const int left = g.N - (p.tiles_n - 1) * p.BN;
        p.nt_tail = std::min(p.BN, (left + 15) / 16 * 16);
        p.idesc_tail = tc::make_idesc_tf32(kBM * p.ctas, p.nt_tail, p.a_mn, p.b_mn);
    }
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = g.C; p.c_si = g.c_si; p.c_sj = g.c_sj; p.c_sb = g.c_sb;
    p.row_bias = g.row_bias; p.relu = g.relu;
    p.Y = g.Y; p.y_ld = g.y_ld; p.y_sb = g.y_bs;
    p.y_split = g.y_split; p.y_group = g.y_group_stride;
    p.err = device_status_ptr();
    if (!p.err) return (int)cudaErrorUnknown;

    CUtensorMap tmA, tmB, tmY, tmR;
    // operand maps: dim0 is the contiguous axis
    {
        const uint64_t rows = (uint64_t)g.M, k = (uint64_t)g.K;
        uint64_t dims[4], str[3];
        uint32_t box[4];
        if (!p.a_mn) { dims[0] = k; dims[1] = rows; box[0] = kBK; box[1] = kBM; }
        else { dims[0] = rows; dims[1] = k; box[0] = 32; box[1] = kBK; }
        dims[2] = p.a_batched ? (uint64_t)g.batch : 1;
        box[2] = 1;
        str[0] = (uint64_t)g.a_ld * 4;
        str[1] = p.a_batched ? (uint64_t)g.a_bs * 4 : str[0] * dims[1];
        dims[3] = 1; box[3] = 1; str[2] = str[1] * dims[2];      // unit dimension: see the producer
        if (!make_tmap(&tmA, g.A, 4, dims, str, box, p.a_mn ? kTmapSwizzle128Atom32 : kTmapSwizzle128))
            return (int)cudaErrorInvalidValue;
    }
    {
        const uint64_t cols = (uint64_t)g.N, k = (uint64_t)g.K;
        uint64_t dims[4], str[3];
        uint32_t box[4];
        if (!p.b_mn) { dims[0] = k; dims[1] = cols; box[0] = kBK; box[1] = (uint32_t)p.BNH; }
        else { dims[0] = cols; dims[1] = k; box[0] = 32; box[1] = kBK; }
        dims[2] = p.b_batched ? (uint64_t)g.batch : 1;
        box[2] = 1;
        str[0] = (uint64_t)g.b_ld * 4;
        str[1] = p.b_batched ? (uint64_t)g.b_bs * 4 : str[0] * dims[1];
        dims[3] = 1; box[3] = 1; str[2] = str[1] * dims[2];
        if (!make_tmap(&tmB, g.B, 4, dims, str, box, p.b_mn ? kTmapSwizzle128Atom32 : kTmapSwizzle128))
            return (int)cudaErrorInvalidValue;
    }
    // MN-major B through one 4-D box per stage: (32 columns, K, blocks of 32 columns, batch).  Only the
    // full blocks of a row belong to the view; a CTA whose columns reach past them loads block by block.
    CUtensorMap tmBb = tmB;
    p.b_big = 0;
    p.b_nblk_full = g.N / 32;
    if (p.b_mn && p.b_nblk_full >= 1 && p.BNH >= 64) {
        uint64_t dims[4] = {32, (uint64_t)g.K, (uint64_t)p.b_nblk_full, p.b_batched ? (uint64_t)g.batch : 1};
        uint64_t str[3] = {(uint64_t)g.b_ld * 4, 128, p.b_batched ? (uint64_t)g.b_bs * 4 : (uint64_t)g.b_ld * 4 * g.K};
        uint32_t box[4] = {32, (uint32_t)kBK, (uint32_t)(p.BNH / 32), 1};
        p.b_big = make_tmap(&tmBb, g.B, 4, dims, str, box, kTmapSwizzle128Atom32) ? 1 : 0;
    }
    if (p.y_tma) {
        uint64_t dims[3] = {(uint64_t)g.N, (uint64_t)g.M, (uint64_t)g.batch};
        uint64_t str[2] = {(uint64_t)g.y_ld * 4, g.batch > 1 ? (uint64_t)g.y_bs * 4 : (uint64_t)g.y_ld * 4 * g.M};
        uint32_t box[3] = {32, 32, 1};
        if (!make_tmap(&tmY, g.Y, 3, dims, str, box, kTmapSwizzle128)) return (int)cudaErrorInvalidValue;
    } else {
        tmY = tmA;   // never dereferenced
    }
    tmR = tmY;
    if (p.r_tma) {
        // the addend has Y's shape and strides, so its view is Y's with another base
        uint64_t dims[3] = {(uint64_t)g.N, (uint64_t)g.M, (uint64_t)g.batch};
        uint64_t str[2] = {(uint64_t)g.y_ld * 4, g.batch > 1 ? (uint64_t)g.y_bs * 4 : (uint64_t)g.y_ld * 4 * g.M};
        uint32_t box[3] = {32, 32, 1};
        if ((reinterpret_cast<uintptr_t>(g.residual) & 15) != 0 ||
            !make_tmap(&tmR, g.residual, 3, dims, str, box, kTmapSwizzle128)) {
            p.r_tma = 0;                       // plain loads serve an addend that TMA cannot address
            p.staging_bytes = kStagingBytes;
        }
    }

    const size_t smem = 1024 + (size_t)p.num_stages * p.stage_bytes + p.staging_bytes + kBarrierBytes;
    const cudaError_t attr_err =
        cudaFuncSetAttribute(p.ctas == 2 ? tc_gemm_kernel<2> : tc_gemm_kernel<1>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (attr_err != cudaSuccess) return (int)attr_err;
    const long long total = (long long)p.tiles_m * p.tiles_n * p.batch;
    const int grid = (int)(total < units ? total : units) * p.ctas;
    const cudaError_t le =
        p.ctas == 2 ? launch_pdl_cluster(tc_gemm_kernel<2>, 2, dim3(grid), dim3(kThreads), smem, (cudaStream_t)stream, tmA,
                                         tmB, tmBb, tmY, tmR, p)
                    : launch_pdl(tc_gemm_kernel<1>, dim3(grid), dim3(kThreads), smem, (cudaStream_t)stream, tmA, tmB, tmBb,
                                 tmY, tmR, p);
    count_launch();
    return (int)le;
}

}  // namespace onnxb
