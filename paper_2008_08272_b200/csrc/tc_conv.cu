// Implicit-GEMM convolution on the tcgen05 tensor cores (TF32 multiply, fp32 accumulate)
// for ONNX Conv (Sec. 4.1) with any kernel size, stride, dilation, padding and groups.
//
// GEMM view: rows = output pixels ("anchors" in slot space, see tc_conv_plan.h), columns =
// output channels, reduction = input channels x filter taps.  The im2col matrix is never
// formed; per block of KB input channels
//   warp 0      stages the raw NCHW rows the tile touches into shared memory by TMA
//               (zero fill outside the tensor);
//   warps 4-11  re-lay them into the K-major "4 channels x slot" operand layout of the MMA,
//               rounding fp32 to TF32 (nearest) and writing zeros for padding;
//   warp 1      streams the pre-packed, pre-rounded weights by bulk copy;
//   warp 2      issues, for every tap, tcgen05.mma on the SAME activation tile at a start address
//               shifted by the tap's slot offset, accumulating in TMEM;
//   warps 12-19 read finished accumulators back (tcgen05.ld), add bias, apply Relu and store NCHW
//               with lanes along consecutive pixels (coalesced); when a tile's accumulators fill at
//               most half of TMEM it holds two sets, so this overlaps the next tile's MMAs.
// CTA pairs (kCtas = 2): two CTAs of a cluster share one tile of 2 x MT x 128 pixels.  Each stages
// its own pixels and HALF of the tile's weight rows; the even CTA issues cta_group::2 MMAs
// (M = 256) that read both CTAs' shared memory and write each CTA's rows into its own TMEM.  Per
// CTA this halves the weight bytes fetched from L2 and the weight bytes the tensor pipe reads from
// shared memory per flop, the two limits of the single-CTA form.  Stage hand-over: the odd CTA's
// epilogue warps arrive directly on the even CTA's barriers, its MMA warp forwards "my weights have
// landed", its relay warp (warp 3) "my operand stage is written", and stage releases come back by
// multicast commit.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "common.h"
#define ONNXB_DEBUG_HOOKS_CONV
#include "debug_hooks.cuh"
#include "tc_common.cuh"
#include "tc_conv_plan.h"
#include "tc_host.h"

namespace onnxb {

namespace {

using namespace tc;

// Warps: raw producer, weight producer, MMA issuer, relay, 8 transform warps, then kEpi (8 or 4) epilogue
// warps.  With 8 epilogue warps the block has 640 threads and 96 registers per thread; with 4 it has 512
// and 128, which the transform warps (ten independent address chains, twenty values in flight) turn into
// speed: layers bound by the transform and with several tiles per CTA (so that the slower epilogue
// hides behind the next tile) take the 4-warp form.
constexpr int kXformWarps = 8;
constexpr int kXformThreads = kXformWarps * 32;
constexpr int kRelayWarp = 3;               // odd CTA of a pair: passes "operand stage written" on to the issuing CTA
constexpr int kFirstXformWarp = 4, kFirstEpiWarp = kFirstXformWarp + kXformWarps;
constexpr int threads_for(int epi_warps) { return (kFirstEpiWarp + epi_warps) * 32; }
constexpr int kOwned = 10;                 // (slot, chunk) units of an A stage one transform thread may own
constexpr int kMaxRawStages = 4;
constexpr int kMaxAStages = 3;
constexpr int kMaxSpb = 8;                 // K-steps per weight stage (the MMA issue loop is unrolled over them)
constexpr int kMaxBStages = 12;
constexpr int kSmemLimit = 232448;
constexpr int kBarBytes = 512;
constexpr int kSegBytes = 256;             // >= sizeof(TcConvSegs)
static_assert(sizeof(TcConvSegs) <= kSegBytes, "segment table does not fit its slot");

struct Bars {
    uint64_t raw_full[kMaxRawStages], raw_empty[kMaxRawStages], a_full[kMaxAStages], a_empty[kMaxAStages];
    uint64_t a_done[kMaxAStages];            // odd CTA of a pair: its transform warps have written the stage
    uint64_t b_full[kMaxBStages], b_empty[kMaxBStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t seg_full[2], seg_empty[2];      // segment tables, one per tile parity
    uint32_t tmem_holder;
};
static_assert(sizeof(Bars) <= kBarBytes, "barrier block too large");

// ------------------------------------------------------------------ weight packing
// Packed layout: [group][channel tile][CTA of the pair][channel block][K-step][chunk 0/1][row BNH][4],
// i.e. for each K-step the exact shared-memory image of one CTA's part of the K-major B operand: two
// 16-byte chunks (4 reduction terms each) per output channel, rows 16 bytes apart.  Values are rounded to TF32 (nearest);
// rows past the group's channels, channels past Cg and unpaired taps are zero.
// Launched with programmatic stream serialization: it may become resident while the previous kernel
// of the stream drains, and waits (pdl_wait) before it touches W or the workspace.
__global__ void pack_weights_kernel(const TcConvPlan g, const float *__restrict__ W, float4 *__restrict__ out) {
    pdl_launch_dependents();
    const unsigned total = (unsigned)(g.packed_floats / 4);          // the planner keeps this below 2^31
    pdl_wait();
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        unsigned t = i;
        const int row = (int)(t % (unsigned)g.BNH); t /= (unsigned)g.BNH;
        const int k = (int)(t & 1u); t >>= 1;
        const int step = (int)(t % (unsigned)g.n_steps); t /= (unsigned)g.n_steps;
        const int cb = (int)(t % (unsigned)g.ncb); t /= (unsigned)g.ncb;
        const unsigned cts = (unsigned)(g.ctiles * g.ctas);
        const int ct = (int)(t % cts); t /= cts;                     // BNH-wide tile: (tile, CTA of the pair)
        const int grp = (int)t;
        const int mg = ct * g.BNH + row;
        const int tap = g.src_tap[step][k];
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (mg < g.Mg && tap >= 0) {
            const int m = grp * g.Mg + mg;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = cb * g.KB + g.src_c0[step][k] + e;
                CHK(((size_t)m * g.Cg + (c < g.Cg ? c : 0)) * g.taps + tap < (size_t)g.M * g.Cg * g.taps, 1, ((size_t)m * g.Cg + c) * g.taps + tap)
                if (c < g.Cg) v[e] = round_tf32(__ldg(W + ((size_t)m * g.Cg + c) * g.taps + tap));
            }
        }
        out[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

// Channel blocks are summed in a rotated order that differs from tile to tile: CTAs working at the
// same time then stream different parts of the (shared) packed weights, instead of all asking the
// same L2 lines at the same moment.
__device__ __forceinline__ int cb_rotation(long long tile, int ncb) { return (int)((tile * 5 + 3) % ncb); }

// ------------------------------------------------------------------ main kernel
// kAdd: the epilogue also adds a tensor laid out like Y (a residual connection) before the Relu.  A
// separate instantiation, so that the plain kernel's register allocation is not disturbed.
// kEpiWarps: 8 or 4 epilogue warps (see the thread layout above).
template <int kCtas, bool kAdd, int kEpiWarps>
__global__ void __launch_bounds__(threads_for(kEpiWarps), 1)
tc_conv_kernel(const __grid_constant__ CUtensorMap tmX, const TcConvPlan g, const float *__restrict__ X,
               const float *__restrict__ Wpk, const float *__restrict__ bias, const float *__restrict__ R,
               float *__restrict__ Y, unsigned int *err) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment by pointer arithmetic on the shared array itself, so that the compiler
    // keeps treating everything derived from it as shared memory (LDS/STS, not generic accesses)
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *a_st = smem;
    uint8_t *raw_st = a_st + (size_t)g.na_stages * g.a_stage_bytes;
    uint8_t *b_st = raw_st + (size_t)g.nr_stages * g.raw_stage_bytes;
    uint8_t *seg_st = b_st + (size_t)g.nb_stages * g.b_stage_bytes;
    Bars *bars = reinterpret_cast<Bars *>(seg_st + kMaxRawStages * kSegBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) LOG(8, 0);
    const int tile_rows = g.MT * 128;
    // CTA pair: rank within the cluster, and the tiles this CTA (pair) walks
    const uint32_t rank = kCtas == 2 ? cluster_ctarank() : 0u;
    const long long first_tile = blockIdx.x / kCtas, tile_step = gridDim.x / kCtas;
    const int cgt = g.ctiles * g.group;        // channel tiles over all groups
    // accumulator placement in TMEM: two alternating sets when one set fits in 256 columns
    const bool acc_dbl = g.MT == 1 || g.BN <= 128;
    const uint32_t mt_cols = acc_dbl ? 128u : 256u;     // column distance between a CTA's two accumulators

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.nr_stages; ++s) {
            mbar_init(&bars->raw_full[s], 1);
            mbar_init(&bars->raw_empty[s], kXformWarps);
        }
        for (int s = 0; s < g.na_stages; ++s) {
            // waited on by the issuing CTA only: its own transform warps, plus one message from the peer
            mbar_init(&bars->a_full[s], kCtas == 2 ? (g.relay ? kXformWarps + 1 : 2 * kXformWarps) : kXformWarps);
            mbar_init(&bars->a_done[s], kXformWarps);
            mbar_init(&bars->a_empty[s], 1);
        }
        for (int s = 0; s < g.nb_stages; ++s) {
            // issuing CTA of a pair: its own producer plus the peer's "landed" message
            mbar_init(&bars->b_full[s], (kCtas == 2 && rank == 0) ? 2 : 1);
            mbar_init(&bars->b_empty[s], 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->acc_full[s], 1);
            mbar_init(&bars->acc_empty[s], kEpiWarps * kCtas);
            mbar_init(&bars->seg_full[s], 1);
            mbar_init(&bars->seg_empty[s], kXformWarps);
        }
        mbar_fence_init();
        if (g.raw_mode == 0) prefetch_tmap(&tmX);
    }
    if (warp == 2) {
        tmem_alloc(&bars->tmem_holder, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_holder;
    if (kCtas == 2) cluster_sync_all();     // the peer's barriers exist before anything arrives on them
    pdl_launch_dependents();
    // Everything above overlapped the previous kernel's tail, and so does each role's own set-up below:
    // the threads that touch global memory (the two producers, the epilogue warps) wait for the previous
    // kernel just before their first access; the others only ever see what those threads hand them.

    if (warp == 0) {
        // ------------------------------------------------------------ raw activation producer
        if (elect_one()) {
            int rs = 0;
            uint32_t rphase = 0, tile_it = 0;
            const long long HW = (long long)g.H * g.W;
            const long long planes_total = (long long)g.N * g.C;
            const int KB = g.KB, ncb = g.ncb, box_floats = g.KB * g.BOXP;
            for (long long t = first_tile; t < g.total_tiles; t += tile_step) {
                const int ct_all = (int)(t % cgt);
                const int grp = ct_all / g.ctiles;
                const long long G0 = ((t / cgt) * kCtas + rank) * tile_rows;
                // The segment table is the same for every channel block of the tile.  Two tables
                // alternate by tile; the transform warps hand a table back once they have turned it
                // into their per-thread offsets, so it is ready long before the tile's data lands.
                const uint32_t sp = tile_it & 1u;
                mbar_wait(&bars->seg_empty[sp], ((tile_it >> 1) & 1u) ^ 1u, err, 20);
                TcConvSegs *segs = reinterpret_cast<TcConvSegs *>(seg_st + sp * kSegBytes);
                tc_conv_segments(g, G0, *segs);
                mbar_arrive(&bars->seg_full[sp]);
                ++tile_it;
                if (tile_it == 1) {
                    pdl_wait();
                    LOG(8, 1);
                }
                const int nseg = segs->nseg;
                const uint32_t tile_bytes = (uint32_t)segs->total_floats * 4u;
                const int rot = cb_rotation(t, ncb);
                for (int cb = 0; cb < ncb; ++cb) {
                    mbar_wait(&bars->raw_empty[rs], rphase ^ 1, err, 11);
                    LOG(0, cb);
                    float *dst = reinterpret_cast<float *>(raw_st + (size_t)rs * g.raw_stage_bytes);
                    const int cbx = cb + rot < ncb ? cb + rot : cb + rot - ncb;
                    const int c0 = grp * g.Cg + cbx * KB;
                    if (g.raw_mode == 0) {
                        mbar_arrive_expect_tx(&bars->raw_full[rs], tile_bytes);
                        for (int i = 0; i < nseg; ++i) {
                            const int plane0 = (segs->n_first + i) * g.C + c0;
                            const int nbox = segs->nbox[i], f0 = segs->f0[i];
                            float *d = dst + segs->base[i];
                            for (int j = 0; j < nbox; ++j)
                                tma_load_2d(d + j * box_floats, &tmX, &bars->raw_full[rs], f0 + j * g.BOXP, plane0);
                        }
                    } else {
                        // whole-image slabs [channel][H*W]; clip at the end of X
                        uint32_t total = 0;
                        for (int i = 0; i < nseg; ++i) {
                            if (!segs->nbox[i]) continue;
                            long long nch = planes_total - ((long long)(segs->n_first + i) * g.C + c0);
                            if (nch > KB) nch = KB;
                            if (nch > 0) total += (uint32_t)(nch * HW * 4);
                        }
                        mbar_arrive_expect_tx(&bars->raw_full[rs], total);
                        for (int i = 0; i < nseg; ++i) {
                            if (!segs->nbox[i]) continue;
                            const long long plane0 = (long long)(segs->n_first + i) * g.C + c0;
                            long long nch = planes_total - plane0;
                            if (nch > KB) nch = KB;
                            if (nch > 0)
                                bulk_load_1d(dst + segs->base[i], X + plane0 * HW, (uint32_t)(nch * HW * 4),
                                             &bars->raw_full[rs]);
                        }
                    }
                    if (++rs == g.nr_stages) { rs = 0; rphase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ weight producer
        if (elect_one()) {
            int bs = 0;
            uint32_t bphase = 0;
            const long long per_ct = (long long)g.ncb * g.n_steps * g.b_step_bytes;   // bytes per channel tile and CTA
            const int nb = g.nb_stages, ncb = g.ncb, b_steps = g.b_steps, spb = g.spb, n_steps = g.n_steps;
            const uint32_t stage_bytes = (uint32_t)g.b_stage_bytes, step_bytes = (uint32_t)g.b_step_bytes;
            pdl_wait();             // the packed weights may come from the kernel just before this one
            for (long long t = first_tile; t < g.total_tiles; t += tile_step) {
                const int ct_all = (int)(t % cgt);
                const uint8_t *tile_src = reinterpret_cast<const uint8_t *>(Wpk) + (ct_all * kCtas + (int)rank) * per_ct;
                const int rot = cb_rotation(t, ncb);
                for (int cb = 0; cb < ncb; ++cb) {
                    const int cbx = cb + rot < ncb ? cb + rot : cb + rot - ncb;
                    const uint8_t *src = tile_src + (long long)cbx * n_steps * step_bytes;
                    for (int bstep = 0; bstep < b_steps; ++bstep) {
                        const uint32_t bytes = (uint32_t)min(spb, n_steps - bstep * spb) * step_bytes;
                        mbar_wait(&bars->b_empty[bs], bphase ^ 1, err, 12);
                        LOG(1, cb * b_steps + bstep);
                        mbar_arrive_expect_tx(&bars->b_full[bs], bytes);
                        bulk_load_1d(b_st + (size_t)bs * stage_bytes, src, bytes, &bars->b_full[bs]);
                        src += bytes;
                        if (++bs == nb) { bs = 0; bphase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ MMA issuer
        // One thread issues every MMA.  Operands are no-swizzle K-major: rows 16 bytes apart, 8-row
        // groups 128 bytes apart (SBO), the two 16-byte K chunks of one instruction LBO apart.  For
        // A the per-step table holds offset and LBO (a chunk pitch, or the distance between two taps);
        // all descriptor words are precomputed, a step costs a table read and a few adds.
        if (kCtas == 2 && rank != 0) {
            // Odd CTA of a pair: the even CTA issues the MMAs.  Tell it when each of this CTA's weight
            // stages has landed (everything else reaches its barriers directly).
            if (elect_one()) {
                const uint32_t peer_b_full = map_to_cta(smem_u32(&bars->b_full[0]), 0);
                const int ncb = g.ncb, nb = g.nb_stages, b_steps = g.b_steps;
                int bs = 0;
                uint32_t bphase = 0;
                for (long long t = first_tile; t < g.total_tiles; t += tile_step) {
                    for (int i = 0; i < ncb * b_steps; ++i) {
                        mbar_wait(&bars->b_full[bs], bphase, err, 19);
                        mbar_arrive_remote(peer_b_full + (uint32_t)bs * 8u);
                        if (++bs == nb) { bs = 0; bphase ^= 1; }
                    }
                }
            }
        } else if (elect_one()) {
            const uint32_t desc_hi = (128u >> 4) | (1u << 14);                 // SBO = 128, descriptor version 1
            const uint32_t a_base16 = (smem_u32(a_st) >> 4) & 0x3FFFu;
            const uint32_t b_lo0 = ((smem_u32(b_st) >> 4) & 0x3FFFu) | (((uint32_t)g.BNH * 16u >> 4) << 16);
            const uint32_t a_stage16 = (uint32_t)g.a_stage_bytes >> 4, b_stage16 = (uint32_t)g.b_stage_bytes >> 4;
            const uint32_t b_step16 = (uint32_t)g.b_step_bytes >> 4;
            const uint32_t idesc = g.idesc;
            const int n_steps = g.n_steps, ncb = g.ncb, nb = g.nb_stages, spb = g.spb, b_steps = g.b_steps;
            const bool two = g.MT == 2;
            int as = 0, bs = 0;
            uint32_t aphase = 0, bphase = 0, it = 0;
            PROF_DECL;
            for (long long t = first_tile; t < g.total_tiles; t += tile_step, ++it) {
                const uint32_t ab = acc_dbl ? (it & 1u) : 0u, use = acc_dbl ? (it >> 1) : it;
                const uint32_t d0 = tmem_base + ab * 256u, d1 = d0 + mt_cols;
                if (kCtas == 2) mbar_wait_cluster(&bars->acc_empty[ab], (use & 1u) ^ 1u, err, 13);
                else mbar_wait(&bars->acc_empty[ab], (use & 1u) ^ 1u, err, 13);
                tc_fence_after_sync();
                PROF_MARK(0);
                uint32_t accumulate = 0;
                for (int cb = 0; cb < ncb; ++cb) {
                    if (kCtas == 2) mbar_wait_cluster(&bars->a_full[as], aphase, err, 14);
                    else mbar_wait(&bars->a_full[as], aphase, err, 14);
                    PROF_MARK(1);
                    LOG(2, cb);
                    const uint32_t a_lo = a_base16 + (uint32_t)as * a_stage16;
                    for (int bstep = 0; bstep < b_steps; ++bstep) {
                        if (kCtas == 2) mbar_wait_cluster(&bars->b_full[bs], bphase, err, 15);
                        else mbar_wait(&bars->b_full[bs], bphase, err, 15);
                        tc_fence_after_sync();
                        PROF_MARK(2);
                        LOG(3, cb * b_steps + bstep);
                        // One thread issues everything, so every dependent instruction here costs
                        // its full latency: fetch the stage's table entries together, then issue
                        // the MMAs back to back with nothing but adds in between.
                        const int s0 = bstep * spb, cnt = min(n_steps - s0, spb);
                        const uint32_t bl = b_lo0 + (uint32_t)bs * b_stage16;
                        uint32_t sa[kMaxSpb];
#pragma unroll
                        for (int j = 0; j < kMaxSpb; ++j) sa[j] = j < cnt ? g.step_a[s0 + j] : 0u;
#pragma unroll
                        for (int j = 0; j < kMaxSpb; ++j) {
                            if (j < cnt) {
                                const uint32_t al = a_lo + sa[j], blj = bl + (uint32_t)j * b_step16;
                                if (kCtas == 2) {
                                    mma_tf32_lohi_pair(d0, al, desc_hi, blj, desc_hi, idesc, accumulate);
                                    if (two) mma_tf32_lohi_pair(d1, al + 128u, desc_hi, blj, desc_hi, idesc, accumulate);
                                } else {
                                    mma_tf32_lohi(d0, al, desc_hi, blj, desc_hi, idesc, accumulate);
                                    if (two) mma_tf32_lohi(d1, al + 128u, desc_hi, blj, desc_hi, idesc, accumulate);
                                }
                                accumulate = 1;
                            }
                        }
                        if (kCtas == 2) mma_commit_pair(&bars->b_empty[bs]);
                        else mma_commit(&bars->b_empty[bs]);
                        if (++bs == nb) { bs = 0; bphase ^= 1; }
                        PROF_MARK(3);
                    }
                    if (kCtas == 2) mma_commit_pair(&bars->a_empty[as]);
                    else mma_commit(&bars->a_empty[as]);
                    LOG(4, cb);
                    if (++as == g.na_stages) { as = 0; aphase ^= 1; }
                }
                if (kCtas == 2) mma_commit_pair(&bars->acc_full[ab]);
                else mma_commit(&bars->acc_full[ab]);
                PROF_MARK(4);
            }
            PROF_FLUSH(0);
        }
    } else if (warp == kRelayWarp) {
        // ------------------------------------------------------------ operand-stage relay (odd CTA of a pair)
        // The issuing CTA's tensor core reads this CTA's operand stage, so the transform warps' writes must
        // be released at cluster scope before the issuing CTA hears of them.  That fence stalls its thread
        // for about a thousand cycles; done by each transform warp it cost them a quarter of their time.
        // They arrive on a barrier of their own CTA instead (CTA scope: cheap), and this thread, which has
        // nothing else to do, acquires that, fences at cluster scope (release is cumulative: it covers what
        // it acquired) and arrives on the issuing CTA's barrier.
        if (kCtas == 2 && rank != 0 && g.relay && elect_one()) {
            const uint32_t peer_a_full = map_to_cta(smem_u32(&bars->a_full[0]), 0);
            const int ncb = g.ncb, na = g.na_stages;
            int as = 0;
            uint32_t aphase = 0;
            for (long long t = first_tile; t < g.total_tiles; t += tile_step) {
                for (int cb = 0; cb < ncb; ++cb) {
                    mbar_wait(&bars->a_done[as], aphase, err, 22);
                    mbar_arrive_remote_release(peer_a_full + (uint32_t)as * 8u);
                    if (++as == na) { as = 0; aphase ^= 1; }
                }
            }
        }
    } else if (warp < kFirstEpiWarp) {
        // ------------------------------------------------------------ transform warps
        const int xw = warp - kFirstXformWarp;     // 0..7
        const int xt = xw * 32 + lane;             // 0..255
        const int cp = g.raw_mode == 1 ? g.H * g.W : g.BOXP;    // channel pitch inside the raw stage
        const int per_stage_slots = g.planes * g.SLOTS;
        const int nchunks = g.nchunks, KB = g.KB, ncb = g.ncb, box_floats = g.KB * g.BOXP, nr = g.nr_stages;
        // Work units: one (slot, 4-channel chunk) pair = four raw reads and one 16-byte operand row.
        // Unit u = chunk * slots + slot; this thread owns units xt, xt + 256, ...
        const int units = per_stage_slots * nchunks;
        const int nu = (units - xt + kXformThreads - 1) / kXformThreads;
        int rs = 0, as = 0;
        uint32_t rphase = 0, aphase = 0, tile_it = 0;
        PROF_DECL;
        const uint32_t a_full_addr = kCtas == 2 ? map_to_cta(smem_u32(&bars->a_full[0]), 0) : 0u;
        // What does not depend on the tile is worked out once: where a unit's operand row goes, and
        // which slot of which parity plane it reads.
        uint32_t udst[kOwned];                     // byte offset of the unit's operand row inside an A stage | chunk index
        // plane << 28 | the slot's place in the stage: as slot rows << 12 | slot columns from the tile's first
        // slot (4 epilogue warps), or as the plain slot index (8)
        uint32_t ujp[kOwned];
#pragma unroll
        for (int i = 0; i < kOwned; ++i) {
            udst[i] = 0;
            ujp[i] = 0;
            if (i < nu) {
                const int u = xt + i * kXformThreads;
                const int ch = conv_fdiv(u, g.planes * g.SLOTS, g.dv_pss), idx = u - ch * per_stage_slots;
                // operand rows are 16 bytes apart: the low four bits carry the unit's chunk index
                udst[i] = ((uint32_t)ch * (uint32_t)g.chunk_pitch + (uint32_t)idx * 16u) | (uint32_t)ch;
                const int pl = conv_fdiv(idx, g.SLOTS, g.dv_SLOTS), j = idx - pl * g.SLOTS;
                // the slot's distance from the tile's first slot, as whole slot rows and columns
                // (both below 2^12: a stage holds at most kOwned * 256 slots)
                const int dh = conv_fdiv(j, g.Ws, g.dv_Ws), dw = j - dh * g.Ws;
                ujp[i] = kEpiWarps == 8 ? (uint32_t)j | ((uint32_t)pl << 28)
                                        : (uint32_t)dw | ((uint32_t)dh << 12) | ((uint32_t)pl << 28);
            }
        }
        for (long long t = first_tile; t < g.total_tiles; t += tile_step) {
            const long long G0 = ((t / cgt) * kCtas + rank) * tile_rows;
            int uoff[kOwned];                      // raw float offset of the unit's first channel, -1 = padding
            const int rot = cb_rotation(t, ncb);
            {
                // per-thread offsets of the tile, from its segment table (ready before the data)
                const uint32_t sp = tile_it & 1u;
                mbar_wait(&bars->seg_full[sp], (tile_it >> 1) & 1u, err, 21);
                PROF_MARK(4);
                ++tile_it;
                const TcConvSegs *segs = reinterpret_cast<const TcConvSegs *>(seg_st + sp * kSegBytes);
                const int n0 = segs->n_first, hq0 = segs->hq0, wq0 = segs->wq0;
                if (kEpiWarps == 8) {
                    // 96 registers per thread: one unit after the other, each leaving early where it can
#pragma unroll
                    for (int i = 0; i < kOwned; ++i) {
                        uoff[i] = -1;
                        if (i < nu) {
                            const int ch = (int)(udst[i] & 15u), pl = (int)(ujp[i] >> 28);
                            const uint32_t Gs = (uint32_t)G0 + (ujp[i] & 0x0FFFFFFFu);     // the planner keeps slots below 2^31
                            if (Gs < (uint32_t)g.total_slots) {
                                const int n = conv_fdiv((int)Gs, g.L, g.dv_L);
                                const int uu = (int)Gs - n * g.L;
                                const int hq = conv_fdiv(uu, g.Ws, g.dv_Ws), wq = uu - hq * g.Ws;
                                // fixed-index reads of the parity tables (a dynamic index into kernel
                                // parameters costs an indexed constant load per use)
                                const int pa = pl == 0 ? g.pa[0] : pl == 1 ? g.pa[1] : pl == 2 ? g.pa[2] : g.pa[3];
                                const int pb = pl == 0 ? g.pb[0] : pl == 1 ? g.pb[1] : pl == 2 ? g.pb[2] : g.pb[3];
                                const int h = hq * g.sh + pa - g.pt;
                                const int w = wq * g.sw + pb - g.pl;
                                const int sg = n - segs->n_first;
                                if ((unsigned)h < (unsigned)g.H && (unsigned)w < (unsigned)g.W && (unsigned)sg < (unsigned)segs->nseg) {
                                    const int f = h * g.W + w - segs->f0[sg];
                                    int o;
                                    if (g.raw_mode == 1) o = segs->base[sg] + f;
                                    else {
                                        const int bx = conv_fdiv(f, g.BOXP, g.dv_BOXP);
                                        o = segs->base[sg] + bx * box_floats + (f - bx * g.BOXP);
                                    }
                                    uoff[i] = o + ch * 4 * cp;
                                }
                            }
                        }
                    }
                } else {
                    // Straight-line code, no branches: the units' chains of dependent integer operations then
                    // overlap instead of running one after the other (this loop, not the data movement, was
                    // the larger part of the thin first layer's time when every unit took its own branches).
                    const int nseg = segs->nseg;
    #pragma unroll
                    for (int i = 0; i < kOwned; ++i) {
                        const int ch = (int)(udst[i] & 15u), pl = (int)(ujp[i] >> 28);
                        // Slot -> (image, slot row, slot column) without dividing the slot number: the tile's
                        // first slot was decomposed once (by the producer, in the segment table); this unit
                        // lies a fixed number of slot rows and columns further on.
                        int wq = wq0 + (int)(ujp[i] & 0xFFFu);
                        const int carry = wq >= g.Ws ? 1 : 0;
                        wq -= carry ? g.Ws : 0;
                        int hq = hq0 + (int)((ujp[i] >> 12) & 0xFFFu) + carry;
                        const int k = conv_fdiv(hq, g.Hs, g.dv_Hs);           // images crossed (small images: several)
                        hq -= k * g.Hs;
                        // fixed-index reads of the parity tables (a dynamic index into kernel parameters
                        // costs an indexed constant load per use)
                        const int pa = pl == 0 ? g.pa[0] : pl == 1 ? g.pa[1] : pl == 2 ? g.pa[2] : g.pa[3];
                        const int pb = pl == 0 ? g.pb[0] : pl == 1 ? g.pb[1] : pl == 2 ? g.pb[2] : g.pb[3];
                        const int h = hq * g.sh + pa - g.pt;
                        const int w = wq * g.sw + pb - g.pl;
                        const bool ok = i < nu && n0 + k < g.N && (unsigned)h < (unsigned)g.H && (unsigned)w < (unsigned)g.W &&
                                        k < nseg;
                        const int sg = k < nseg ? k : 0;                      // a table entry that exists, whatever k is
                        const int f = h * g.W + w - segs->f0[sg];
                        int o = segs->base[sg] + f;                           // whole-image slabs
                        if (g.raw_mode != 1) {
                            const int bx = g.boxp_shift >= 0 ? (f >> g.boxp_shift) : conv_fdiv(ok ? f : 0, g.BOXP, g.dv_BOXP);
                            o = segs->base[sg] + bx * box_floats + (f - bx * g.BOXP);
                        }
                        uoff[i] = ok ? o + ch * 4 * cp : -1;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->seg_empty[sp]);
                PROF_MARK(5);
            }
            for (int cb = 0; cb < ncb; ++cb) {
                mbar_wait(&bars->raw_full[rs], rphase, err, 16);
                PROF_MARK(0);
                if (xt == 0) LOG(5, cb);
                mbar_wait(&bars->a_empty[as], aphase ^ 1, err, 17);
                PROF_MARK(1);
                if (xt == 0) LOG(6, cb);
                const float *raw = reinterpret_cast<const float *>(raw_st + (size_t)rs * g.raw_stage_bytes);
                uint8_t *adst = a_st + (size_t)as * g.a_stage_bytes;
                const int cbx = cb + rot < ncb ? cb + rot : cb + rot - ncb;
                const int c_left = g.Cg - cbx * KB;    // channels of this block that exist
                // In two batches of five units: all reads of a batch first (independent, so their latencies
                // overlap), then round and store; channels past the end of the group (last block only)
                // read as zero.
#pragma unroll
                for (int h0 = 0; h0 < kOwned; h0 += kOwned / 2) {
                    float v[kOwned / 2][4];
#pragma unroll
                    for (int k = 0; k < kOwned / 2; ++k) {
                        const int i = h0 + k;
                        v[k][0] = v[k][1] = v[k][2] = v[k][3] = 0.f;
                        if (i < nu && uoff[i] >= 0) {
                            const float *r = raw + uoff[i];
                            const int left = c_left - (int)(udst[i] & 15u) * 4;
                            if (left > 0) v[k][0] = r[0];
                            if (left > 1) v[k][1] = r[cp];
                            if (left > 2) v[k][2] = r[2 * cp];
                            if (left > 3) v[k][3] = r[3 * cp];
                        }
                    }
#pragma unroll
                    for (int k = 0; k < kOwned / 2; ++k) {
                        const int i = h0 + k;
                        if (i < nu)
                            *reinterpret_cast<float4 *>(adst + (udst[i] & ~15u)) =
                                make_float4(round_tf32(v[k][0]), round_tf32(v[k][1]), round_tf32(v[k][2]),
                                            round_tf32(v[k][3]));
                    }
                }
                PROF_MARK(2);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (kCtas == 2 && rank != 0) {
                        if (g.relay) mbar_arrive(&bars->a_done[as]);                // the relay warp passes it on
                        else mbar_arrive_remote_release(a_full_addr + (uint32_t)as * 8u);
                    } else {
                        mbar_arrive(&bars->a_full[as]);                             // the issuing CTA's own barrier
                    }
                    mbar_arrive(&bars->raw_empty[rs]);
                }
                PROF_MARK(3);
                if (xt == 0) LOG(7, cb);
                if (++rs == nr) { rs = 0; rphase ^= 1; }
                if (++as == g.na_stages) { as = 0; aphase ^= 1; }
            }

        }
        if (xt == 0) PROF_FLUSH(5);
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int ew = warp - kFirstEpiWarp;       // 0..7
        const int quarter = warp & 3;              // TMEM lane quarter this warp may read
        const long long PQ = (long long)g.P * g.Q;
        const bool two = g.MT == 2;
        const uint32_t acc_empty_addr = kCtas == 2 ? map_to_cta(smem_u32(&bars->acc_empty[0]), 0) : 0u;
        uint32_t it = 0;
        for (long long t = first_tile; t < g.total_tiles; t += tile_step, ++it) {
            const int ct_all = (int)(t % cgt);
            const int grp = ct_all / g.ctiles, ct = ct_all % g.ctiles;
            const long long G0 = ((t / cgt) * kCtas + rank) * tile_rows;
            const uint32_t ab = acc_dbl ? (it & 1u) : 0u, use = acc_dbl ? (it >> 1) : it;
            mbar_wait(&bars->acc_full[ab], use & 1u, err, 18);
            tc_fence_after_sync();
            if (it == 0) pdl_wait();        // long since satisfied: the producers passed theirs before the first load
            if (ew == 0 && lane == 0) LOG(8, 2);
            const int nch = (g.BN + 31) / 32;
            // eight warps: two per TMEM lane quarter, each taking half of the tile; four: one per quarter, both halves
            for (int hf = ew >> 2; hf < 2; hf += kEpiWarps / 4) {
            int mt, ch_lo, ch_hi;
            if (two) { mt = hf; ch_lo = 0; ch_hi = nch; }
            else { mt = 0; ch_lo = hf ? (nch + 1) / 2 : 0; ch_hi = hf ? nch : (nch + 1) / 2; }
            const uint32_t acc_col = ab * 256u + (uint32_t)mt * mt_cols;
            const uint32_t G = (uint32_t)G0 + (uint32_t)(mt * 128 + quarter * 32 + lane);
            bool valid = G < (uint32_t)g.total_slots;
            float *yrow = Y;
            if (valid) {
                const int n = (int)(G / (uint32_t)g.L);
                const int u = (int)(G - (uint32_t)n * (uint32_t)g.L);
                const int p = u / g.Ws, q = u - p * g.Ws;
                valid = p < g.P && q < g.Q;
                yrow = Y + ((long long)n * g.M * g.P + p) * g.Q + q;
            }
            const int m_lim = min(g.Mg, (ct + 1) * g.BN);          // channels of this tile that exist
            for (int chunk = ch_lo; chunk < ch_hi; ++chunk) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc_col + (uint32_t)(chunk * 32), v);
                const int mg0 = ct * g.BN + chunk * 32;            // first channel (within the group) of the chunk
                // lane j fetches the bias of column j once; columns then take it by shuffle
                const float bl = (bias && mg0 + lane < m_lim) ? __ldg(bias + grp * g.Mg + mg0 + lane) : 0.f;
                float *yp = yrow + (long long)(grp * g.Mg + mg0) * PQ;
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float x = __uint_as_float(v[j]) + __shfl_sync(0xffffffffu, bl, j);
                    const bool live = valid && mg0 + j < m_lim;
                    if (kAdd && live) x += __ldg(R + (yp - Y));             // residual addend at Y's own position
                    if (g.relu) x = fmaxf(x, 0.f);
                    if (live) *yp = x;
                    yp += PQ;
                }
            }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (ew == 0 && lane == 0) LOG(8, 3);
            if (lane == 0) {
                if (kCtas == 2) mbar_arrive_remote(acc_empty_addr + ab * 8u);
                else mbar_arrive(&bars->acc_empty[ab]);
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (kCtas == 2) cluster_sync_all();     // no CTA leaves while its peer may still signal it
    if (threadIdx.x == 0) LOG(8, 4);
    if (warp == 2) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------ planning (host)
struct Axis {
    int E, Amax, npar, par[kConvMaxPlanes];
};

// Slot extent along one axis: input size I, output size O, leading pad, stride s, dilation d, kernel k.
bool plan_axis(int I, int O, int pad, int s, int d, int k, Axis &ax) {
    int offmax[64];
    bool used[64];
    if (s > 64) return false;
    for (int a = 0; a < s; ++a) { used[a] = false; offmax[a] = 0; }
    ax.Amax = 0;
    for (int t = 0; t < k; ++t) {
        const int a = (t * d) % s, o = (t * d) / s;
        used[a] = true;
        offmax[a] = std::max(offmax[a], o);
        ax.Amax = std::max(ax.Amax, o);
    }
    ax.npar = 0;
    int a_min = -1;
    long long e = O;
    for (int a = 0; a < s; ++a) {
        if (!used[a]) continue;
        if (ax.npar == kConvMaxPlanes) return false;
        ax.par[ax.npar++] = a;
        if (a_min < 0) a_min = a;
        const int z = pad > a ? (pad - a + s - 1) / s : 0;         // leading zero slots of this parity
        e = std::max<long long>(e, (long long)O + offmax[a] - z);
    }
    e = std::max<long long>(e, ((long long)I + pad - a_min + s - 1) / s);
    e = std::min<long long>(e, (long long)O + ax.Amax);
    ax.E = (int)e;
    return true;
}

int pick_conv_bn(int Mg) {
    if (Mg <= 256) return (Mg + 15) / 16 * 16;
    int best = 256, best_pad = 1 << 30;
    for (int bn : {256, 192, 128}) {
        const int padded = (Mg + bn - 1) / bn * bn;
        if (padded < best_pad) { best_pad = padded; best = bn; }
    }
    return best;
}

bool fill_plan(const ConvGeom &c, int ctas, int MT, int BN, int KB, TcConvPlan &g) {
    if (ctas == 2 && BN % 16) return false;      // M = 256 instructions take N in multiples of 16
    g.ctas = ctas;
    g.BNH = BN / ctas;
    g.N = c.N; g.C = c.C; g.H = c.H; g.W = c.W; g.M = c.M; g.Cg = c.Cg; g.Mg = c.Mg;
    g.kH = c.kH; g.kW = c.kW; g.P = c.P; g.Q = c.Q; g.pt = c.pt; g.pl = c.pl;
    g.sh = c.sh; g.sw = c.sw; g.dh = c.dh; g.dw = c.dw; g.group = c.group; g.relu = c.relu;
    g.taps = c.kH * c.kW;
    if (g.taps > kConvMaxTaps) return false;
    Axis ah, aw;
    if (!plan_axis(c.H, c.P, c.pt, c.sh, c.dh, c.kH, ah)) return false;
    if (!plan_axis(c.W, c.Q, c.pl, c.sw, c.dw, c.kW, aw)) return false;
    if (ah.npar * aw.npar > kConvMaxPlanes) return false;
    g.Hs = ah.E; g.Ws = aw.E;
    const long long L = (long long)g.Hs * g.Ws;
    if (L > (1 << 24)) return false;
    g.L = (int)L;
    g.total_slots = (long long)c.N * L;
    if (g.total_slots + 4096 >= (1LL << 31)) return false;        // device code indexes slots in 32 bits
    g.planes = 0;
    for (int i = 0; i < ah.npar; ++i)
        for (int j = 0; j < aw.npar; ++j) { g.pa[g.planes] = ah.par[i]; g.pb[g.planes] = aw.par[j]; ++g.planes; }
    g.a_min = ah.par[0]; g.a_max = ah.par[ah.npar - 1];
    const long long maxshift = (long long)ah.Amax * g.Ws + aw.Amax;
    g.MT = MT; g.BN = BN;
    g.ctiles = (c.Mg + BN - 1) / BN;
    const long long slots = (long long)MT * 128 + maxshift;
    if (c.Cg < 16) KB = 4;
    if (slots * g.planes * (KB / 4) > kOwned * kXformThreads) return false;
    g.SLOTS = (int)slots;
    if ((g.SLOTS + L - 2) / L + 1 > kConvMaxSeg) return false;
    g.plane_pitch = g.SLOTS * 16;
    g.chunk_pitch = g.planes * g.plane_pitch;
    if (g.chunk_pitch >= (1 << 18)) return false;

    // per-tap plane and slot shift, in 16-byte units inside an A stage
    int tap_plane[kConvMaxTaps], tap_off16[kConvMaxTaps];
    for (int r = 0; r < c.kH; ++r)
        for (int s = 0; s < c.kW; ++s) {
            const int a = (r * c.dh) % c.sh, b = (s * c.dw) % c.sw;
            int pl = 0;
            while (g.pa[pl] != a || g.pb[pl] != b) ++pl;
            const int shift = ((r * c.dh) / c.sh) * g.Ws + (s * c.dw) / c.sw;
            tap_plane[r * c.kW + s] = pl;
            tap_off16[r * c.kW + s] = (pl * g.plane_pitch + shift * 16) >> 4;
        }

    // K-steps of one channel block
    if (c.Cg >= 16) {
        // blocks of KB = 16, 32 or 64 channels: KB/8 steps per tap, step j reading chunks 2j and 2j+1
        const int spt = KB / 8;
        g.KB = KB;
        g.n_steps = spt * g.taps;
        if (g.n_steps > kConvMaxSteps) return false;
        const uint32_t lbo16 = (uint32_t)g.chunk_pitch >> 4;
        if ((uint32_t)(KB / 4) * lbo16 >= (1u << 14)) return false;     // every chunk start must fit the address field
        for (int tp = 0; tp < g.taps; ++tp)
            for (int j = 0; j < spt; ++j) {
                const int s = spt * tp + j;
                g.step_a[s] = ((uint32_t)tap_off16[tp] + (uint32_t)j * 2u * lbo16) | (lbo16 << 16);
                g.src_tap[s][0] = g.src_tap[s][1] = (short)tp;
                g.src_c0[s][0] = (short)(j * 8);
                g.src_c0[s][1] = (short)(j * 8 + 4);
            }
    } else {
        // tap pairs: within each plane, taps in order of their offset, two per step
        g.KB = 4;
        g.n_steps = 0;
        for (int pl = 0; pl < g.planes; ++pl) {
            int list[kConvMaxTaps], n = 0;
            for (int tp = 0; tp < g.taps; ++tp)
                if (tap_plane[tp] == pl) list[n++] = tp;
            std::sort(list, list + n, [&](int x, int y) { return tap_off16[x] < tap_off16[y]; });
            for (int i = 0; i < n; i += 2) {
                const int t0 = list[i], t1 = i + 1 < n ? list[i + 1] : -1;
                const uint32_t lbo16 = t1 >= 0 ? (uint32_t)(tap_off16[t1] - tap_off16[t0]) : 0u;
                if (lbo16 >= (1u << 14)) return false;
                const int s = g.n_steps++;
                g.step_a[s] = (uint32_t)tap_off16[t0] | (lbo16 << 16);
                g.src_tap[s][0] = (short)t0;
                g.src_tap[s][1] = (short)t1;
                g.src_c0[s][0] = g.src_c0[s][1] = 0;
            }
        }
    }
    for (int s = g.n_steps; s < kConvMaxSteps; ++s) {
        g.step_a[s] = 0;
        g.src_tap[s][0] = g.src_tap[s][1] = -1;
        g.src_c0[s][0] = g.src_c0[s][1] = 0;
    }
    g.nchunks = g.KB / 4;
    g.ncb = (c.Cg + g.KB - 1) / g.KB;
    const long long ptiles = (g.total_slots + MT * 128 - 1) / (MT * 128);      // per-CTA pixel tiles
    if (ptiles > 0x7fffffffLL) return false;
    g.pix_tiles = (int)((ptiles + ctas - 1) / ctas);
    g.total_tiles = (long long)g.pix_tiles * g.ctiles * c.group;
    // raw staging mode
    const long long HW = (long long)c.H * c.W;
    if (HW % 4 == 0) {
        g.raw_mode = 0;
    } else if (c.Cg % 4 == 0 && c.C % 4 == 0 && HW * g.KB * 4 <= 32768) {
        g.raw_mode = 1;
    } else {
        return false;
    }
    g.a_stage_bytes = g.nchunks * g.chunk_pitch;
    g.a_stage_bytes = (g.a_stage_bytes + 127) / 128 * 128;
    g.b_step_bytes = g.BNH * 32;
    g.spb = std::max(1, std::min(std::min(g.n_steps, kMaxSpb), 32768 / g.b_step_bytes));   // several K-steps per weight stage
    g.idesc = tc::make_idesc_tf32(128 * ctas, BN, 0, 0);
    g.packed_floats = (long long)c.group * g.ctiles * g.ncb * g.n_steps * BN * 8;     // both CTAs' parts
    if (g.packed_floats >= (1LL << 32)) return false;                                  // 32-bit indexing in the packing kernel
    // raw stage size: widest flat pixel range any tile needs, found by walking the tiles
    g.BOXP = 256;
    const long long walk = std::min<long long>(ptiles, L + 2);
    if (g.raw_mode == 0) {
        int widest = 4;
        for (long long i = 0; i <= walk; ++i) {
            const long long pt = i < walk ? i : ptiles - 1;
            const long long G0 = pt * MT * 128;
            const long long Gend = std::min<long long>(G0 + g.SLOTS, g.total_slots);
            const int n_first = (int)(G0 / L), n_last = (int)((Gend - 1) / L);
            for (int n = n_first; n <= n_last; ++n) {
                const long long lo = std::max<long long>(G0, (long long)n * L), hi = std::min<long long>(Gend, (long long)(n + 1) * L);
                const int hq_lo = (int)((lo - (long long)n * L) / g.Ws), hq_hi = (int)((hi - 1 - (long long)n * L) / g.Ws);
                const int h_min = std::max(0, hq_lo * c.sh + g.a_min - c.pt);
                const int h_max = std::min(c.H - 1, hq_hi * c.sh + g.a_max - c.pt);
                if (h_min > h_max) continue;
                const int f0 = (h_min * c.W) & ~3;
                widest = std::max(widest, (h_max + 1) * c.W - f0);
            }
        }
        // boxes of <= 256 pixels, split evenly; every box must start on a 128-byte boundary of
        // shared memory (TMA destination alignment), i.e. KB * BOXP * 4 bytes is a multiple of 128
        const int align = std::max(4, 32 / g.KB);
        widest = (widest + 3) / 4 * 4;
        const int nbox = (widest + 255) / 256;
        g.BOXP = std::min(256, ((widest + nbox - 1) / nbox + align - 1) / align * align);
        // Blocks of 4 channels (the thin first layer of a network) stage so little per pixel that whole
        // 256-pixel boxes cost nothing, and a power of two spares the transform a division per unit.
        if (g.KB == 4 && widest > 128) g.BOXP = 256;
    }
    {
        int worst = 0;
        TcConvSegs segs;
        for (long long i = 0; i <= walk; ++i) {
            const long long pt = i < walk ? i : ptiles - 1;
            tc_conv_segments(g, pt * MT * 128, segs);
            worst = std::max(worst, segs.total_floats);
        }
        g.raw_stage_bytes = (worst * 4 + 127) / 128 * 128;
        if (g.raw_stage_bytes == 0) g.raw_stage_bytes = 128;
    }
    // Raw stages: a third one (the raw tiles come from L2/HBM with a microsecond of latency) when that
    // still leaves 64 KB for the weight ring.
    g.na_stages = 2;
    g.nr_stages = 2;
    g.relay = 0;
    {
        // "ONNXB_CONV_STAGES=a,r" pins the operand / raw stage counts for A/B measurements
        int fa = 0, fr = 0;
        const char *e = getenv("ONNXB_CONV_STAGES");
        if (e && sscanf(e, "%d,%d", &fa, &fr) == 2 && fa >= 2 && fa <= kMaxAStages && fr >= 2 && fr < kMaxRawStages) {
            g.na_stages = fa;
            g.nr_stages = fr;
        } else if (MT == 2 && g.KB >= 16 &&
                   kSmemLimit - (1024 + 3LL * g.a_stage_bytes + kMaxRawStages * kSegBytes + kBarBytes) -
                           2LL * g.raw_stage_bytes >= 65536) {
            // Two accumulators per CTA: a third operand stage instead of a third raw stage (64 -> 64
            // channels at 56x56: 55.5 -> 52.3 us), and in a CTA pair the odd CTA's "stage written" message
            // through its relay warp.  The message then arrives later, which three stages absorb, and the
            // transform warps no longer wait for their cluster-scope fence (128 -> 128 channels at 28x28:
            // 43.4 -> 41.0 us; with two stages the relay loses).
            g.na_stages = 3;
            g.relay = ctas == 2 ? 1 : 0;
        } else {
            const long long bf = 1024 + 2LL * g.a_stage_bytes + kMaxRawStages * kSegBytes + kBarBytes;
            for (int nr = 3; nr <= kMaxRawStages - 1; ++nr)
                if (kSmemLimit - bf - (long long)nr * g.raw_stage_bytes >= 65536) g.nr_stages = nr;
        }
    }
    const long long base_fixed = 1024 + (long long)g.na_stages * g.a_stage_bytes + kMaxRawStages * kSegBytes + kBarBytes;
    const long long fixed = base_fixed + (long long)g.nr_stages * g.raw_stage_bytes;
    const long long room = kSmemLimit - fixed;
    while (room < 3LL * g.spb * g.b_step_bytes && g.spb > 1) g.spb = (g.spb + 1) / 2;   // keep three stages in flight
    g.b_steps = (g.n_steps + g.spb - 1) / g.spb;
    g.b_stage_bytes = g.spb * g.b_step_bytes;
    if (room < 2LL * g.b_stage_bytes) return false;
    g.nb_stages = (int)std::min<long long>(kMaxBStages, room / g.b_stage_bytes);
    g.dv_L = conv_divisor(g.L);
    g.dv_Ws = conv_divisor(g.Ws);
    g.dv_Hs = conv_divisor(g.Hs);
    g.boxp_shift = -1;
    for (int b = 0; b < 16; ++b)
        if ((1 << b) == g.BOXP) g.boxp_shift = b;
    g.dv_BOXP = conv_divisor(g.BOXP);
    g.dv_SLOTS = conv_divisor(g.SLOTS);
    g.dv_pss = conv_divisor(g.planes * g.SLOTS);
    return true;
}

}  // namespace

bool tc_conv_plan(const ConvGeom &c, TcConvPlan &plan, bool forced) {
    const long long taps = (long long)c.kH * c.kW;
    if (c.Cg < 16) {
        // tap-pair mode needs at least two taps, and is kept for problems big enough to matter:
        // tiny thin contractions (an MNIST-size first layer) stay on the exact fp32 SIMT kernel
        const double flops = 2.0 * c.N * c.M * c.P * c.Q * c.Cg * (double)taps;
        if (taps < 2 || c.Cg * taps < 32 || (flops < 5e7 && !forced)) return false;
    }
    const int sms = 148;
    const int bn0 = pick_conv_bn(c.Mg);
    // candidate tiles (CTAs per tile, accumulators per CTA, channels per tile)
    int cand[48][4];
    int ncand = 0;
    auto add = [&](int ctas, int mt, int bn, int kb) {
        for (int i = 0; i < ncand; ++i)
            if (cand[i][0] == ctas && cand[i][1] == mt && cand[i][2] == bn && cand[i][3] == kb) return;
        cand[ncand][0] = ctas; cand[ncand][1] = mt; cand[ncand][2] = bn; cand[ncand][3] = kb; ++ncand;
    };
    int fc = 0, fm = 0, fb = 0, fk = 16;
    if (const char *e = getenv("ONNXB_CONV_TILE")) {      // "ctas,MT,BN[,KB]": pin the tile for A/B measurements
        if (sscanf(e, "%d,%d,%d,%d", &fc, &fm, &fb, &fk) >= 3 && (fc == 1 || fc == 2) && (fm == 1 || fm == 2) &&
            fb >= 16 && fb <= 256 && fb % 16 == 0 && (fk == 16 || fk == 32 || fk == 64))
            add(fc, fm, fb, fk);
    }
    if (ncand == 0) {
        for (int kb = 16; kb <= 64 && (kb == 16 || kb <= c.Cg); kb *= 2)
            for (int ctas = 2; ctas >= 1; --ctas) {
                add(ctas, 2, bn0, kb);
                add(ctas, 1, bn0, kb);
                if (bn0 > 128) { add(ctas, 2, 128, kb); add(ctas, 1, 128, kb); }
                if (bn0 > 64) add(ctas, 1, 64, kb);
            }
    }
    bool have = false;
    double best_cost = 0;
    for (int i = 0; i < ncand; ++i) {
        TcConvPlan p;
        if (!fill_plan(c, cand[i][0], cand[i][1], cand[i][2], cand[i][3], p)) continue;
        // Cost in SM cycles per CTA, fitted to measured tile sweeps of the ResNet-50 3x3 layers.  Per
        // channel block the slowest of: the tensor pipe (BN/2 cycles per 128 x BN x 8 share of an
        // instruction, or the 128 bytes/cycle of shared memory its operands need, whichever is longer),
        // shared memory as a whole (operand reads plus the stages written and the transform, at about
        // 90 bytes/cycle sustained), the weight stream out of L2 (about 3600 bytes/cycle over all SMs, at
        // most 48 per SM) and the transform warps; plus a fixed hand-over cost per block, larger for
        // pairs (their barriers cross the cluster).
        const int units = sms / p.ctas;                                     // tiles in flight
        const long long waves = (p.total_tiles + units - 1) / units;
        const double active = (double)std::min<long long>(p.total_tiles, units) * p.ctas;
        const double n_inst = (double)p.n_steps * p.MT;
        const double op_bytes = 4096.0 + p.BNH * 32.0;
        const double t_mma = n_inst * (std::max(p.BN / 2.0, op_bytes / 128.0) + (p.ctas == 2 ? 10.0 : 0.0));
        const double w_bytes = (double)p.n_steps * p.b_step_bytes;
        const double slots16 = (double)p.planes * p.SLOTS * 16.0 * p.nchunks;
        const double t_smem = (n_inst * op_bytes + w_bytes + 3.0 * slots16) / 90.0;
        // the weight ring must also cover the latency of its copies (about 2500 cycles from issue to
        // landing under load): a ring holding less than that much of the stream paces the block
        const double ring = (double)p.nb_stages * p.b_stage_bytes;
        const double t_w = std::max(w_bytes / std::min(48.0, 3600.0 / active), w_bytes * 2500.0 / ring);
        const double t_x = 300.0 + 100.0 * ((p.planes * p.SLOTS * p.nchunks + 255) / 256);
        // (three operand stages hide most of the hand-over)
        const double per_cb = std::max(std::max(t_mma, t_smem), std::max(t_w, t_x)) +
                              (p.na_stages == 3 ? 300.0 : 400.0 + (p.ctas == 2 ? 700.0 : 0.0));
        const bool dbl = p.MT == 1 || p.BN <= 128;
        const double t_epi = 8.0 * p.MT * p.BN;                             // read-back and stores of one tile
        const double per_tile = (dbl ? std::max(p.ncb * per_cb, t_epi) : p.ncb * per_cb + t_epi) + 3000.0;
        double cost = (double)waves * per_tile + 9000.0 + (dbl ? t_epi : 0.0);
        // pairs of 64-channel tiles with two accumulators measure 12-15 % slower than this model says
        // (64 -> 64 channels at 56x56: 59 us against 52 us with one CTA per tile)
        if (p.ctas == 2 && p.MT == 2 && p.BN <= 64 && p.KB >= 16) cost *= 1.15;
        // tap-pair mode (thin first layers) streams hardly any weights, so a pair shares nothing worth its
        // hand-over (ResNet-50 stem: 106.8 us as pairs, 101.8 us with one CTA per tile)
        if (p.ctas == 2 && p.KB == 4) cost *= 1.15;
        if (!have || cost < best_cost * 0.999) {
            have = true;
            best_cost = cost;
            plan = p;
        }
    }
    if (have) {
        // Four epilogue warps (and 128 registers per thread) where the transform paces the kernel and a
        // CTA walks several tiles: the tap-pair mode of thin first layers (measured: 116 -> 104 us on the
        // ResNet-50 stem; 16-channel blocks gain nothing).  Pinned by
        // ONNXB_CONV_EPI = 4 | 8 for A/B measurements.
        const int units = sms / plan.ctas;
        plan.epi_warps = (plan.KB == 4 && plan.total_tiles >= 3LL * units) ? 4 : 8;
        if (const char *e = getenv("ONNXB_CONV_EPI"))
            if (e[0] == '4' || e[0] == '8') plan.epi_warps = e[0] - '0';
        // Thin first layers in tap-pair mode are paced by the transform warps: take their fence off them too
        // (ResNet-50 stem: 109.3 -> 106.6 us).  ONNXB_CONV_RELAY = 0 | 1 pins the choice for A/B measurements.
        if (plan.ctas == 2 && plan.KB == 4) plan.relay = 1;
        if (const char *e = getenv("ONNXB_CONV_RELAY"))
            if (e[0] == '0' || e[0] == '1') plan.relay = e[0] - '0';
    }
    return have;
}

// How many CTA pairs (clusters of two) of the pair kernel the device runs at once; queried once.
static int max_pairs() {
    static std::atomic<int> cached{-1};
    int n = cached.load(std::memory_order_acquire);
    if (n >= 0) return n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * 148);
    cfg.blockDim = dim3(threads_for(8));
    cfg.dynamicSmemBytes = kSmemLimit;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc_conv_kernel<2, false, 8>, &cfg) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = tc_host::num_sms() / 2;
    }
    cached.store(n, std::memory_order_release);
    return n;
}

size_t tc_conv_workspace_bytes(const TcConvPlan &plan) { return (size_t)plan.packed_floats * 4; }

int launch_tc_conv(const TcConvPlan &plan, const float *X, const float *W, const float *B, const float *R, float *Y,
                   void *workspace, void *stream, int phase) {
    using namespace tc_host;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned int *err = device_status_ptr();
    if (!err) return (int)cudaErrorUnknown;

    // 1. pack + round the weights into the workspace (skipped when the caller packed them earlier)
    if (phase != kTcConvRunOnly) {
        const long long vec = plan.packed_floats / 4;
        const int blocks = (int)std::min<long long>((vec + 255) / 256, 148 * 16);
        const cudaError_t e = launch_pdl(pack_weights_kernel, dim3(blocks), dim3(256), 0, st, plan, W,
                                         reinterpret_cast<float4 *>(workspace));
        count_launch();
        if (e != cudaSuccess) return (int)e;
    }
    if (phase == kTcConvPackOnly) return 0;
    // 2. the convolution
    CUtensorMap tmX;
    if (plan.raw_mode == 0) {
        const uint64_t dims[2] = {(uint64_t)plan.H * plan.W, (uint64_t)plan.N * plan.C};
        const uint64_t str[1] = {(uint64_t)plan.H * plan.W * 4};
        const uint32_t box[2] = {(uint32_t)plan.BOXP, (uint32_t)plan.KB};
        if (!make_tmap(&tmX, X, 2, dims, str, box, kTmapSwizzleNone)) return (int)cudaErrorInvalidValue;
    } else {
        memset(&tmX, 0, sizeof tmX);
    }
    const size_t smem = 1024 + (size_t)plan.na_stages * plan.a_stage_bytes + (size_t)plan.nr_stages * plan.raw_stage_bytes +
                        (size_t)plan.nb_stages * plan.b_stage_bytes + kMaxRawStages * kSegBytes + kBarBytes;
    const bool pair = plan.ctas == 2;
    const bool add = R != nullptr;
    const bool epi4 = plan.epi_warps == 4;
    auto kern = epi4 ? (pair ? (add ? tc_conv_kernel<2, true, 4> : tc_conv_kernel<2, false, 4>)
                             : (add ? tc_conv_kernel<1, true, 4> : tc_conv_kernel<1, false, 4>))
                     : (pair ? (add ? tc_conv_kernel<2, true, 8> : tc_conv_kernel<2, false, 8>)
                             : (add ? tc_conv_kernel<1, true, 8> : tc_conv_kernel<1, false, 8>));
    const int threads = threads_for(epi4 ? 4 : 8);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return (int)e;
    const int sms = num_sms();
    // persistent: one CTA per SM; pairs are clusters of two neighbouring SMs
    const int units = pair ? max_pairs() : sms;
    if (units < 1) return (int)cudaErrorLaunchOutOfResources;
    const int grid = (int)std::min<long long>(plan.total_tiles, units) * plan.ctas;
#ifdef ONNXB_PROFILE
    fprintf(stderr, "[plan] ctas %d MT %d BN %d ctiles %d SLOTS %d planes %d Hs %d Ws %d L %d KB %d ncb %d steps %d spb %d tiles %lld grid %d raw_mode %d BOXP %d a_stage %d raw_stage %d b_stage %d nb %d smem %zu\n",
            plan.ctas, plan.MT, plan.BN, plan.ctiles, plan.SLOTS, plan.planes, plan.Hs, plan.Ws, plan.L, plan.KB, plan.ncb,
            plan.n_steps, plan.spb, plan.total_tiles, grid, plan.raw_mode, plan.BOXP, plan.a_stage_bytes,
            plan.raw_stage_bytes, plan.b_stage_bytes, plan.nb_stages, smem);
#endif
    const cudaError_t le =
        pair ? launch_pdl_cluster(kern, 2, dim3(grid), dim3(threads), smem, st, tmX, plan, X,
                                  reinterpret_cast<const float *>(workspace), B, R, Y, err)
             : launch_pdl(kern, dim3(grid), dim3(threads), smem, st, tmX, plan, X,
                          reinterpret_cast<const float *>(workspace), B, R, Y, err);
    count_launch();
    return (int)le;
}

}  // namespace onnxb
