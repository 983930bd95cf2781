// Implicit-GEMM convolution on the tcgen05 tensor cores (TF32 multiply, fp32 accumulate)
// for ONNX Conv (Sec. 4.1) with any kernel size, stride, dilation, padding and (wide) groups.
//
// GEMM view: rows = output pixels ("anchors" in slot space, see tc_conv_plan.h), columns =
// output channels, reduction = input channels x filter taps.  The im2col matrix is never
// formed; per block of 16 input channels
//   warp 0      stages the raw NCHW rows the tile touches into shared memory by TMA
//               (zero fill outside the tensor);
//   warps 3-10  re-lay them into the K-major "4 channels x slot" operand layout of the MMA,
//               rounding fp32 to TF32 (nearest) and writing zeros for padding;
//   warp 1      streams the pre-packed, pre-rounded weights of (channel block, tap) by bulk copy;
//   warp 2      issues, for every tap, tcgen05.mma on the SAME activation tile at a start address
//               shifted by the tap's slot offset, accumulating in TMEM;
// then warps 3-10 read the accumulators back (tcgen05.ld), add bias, apply Relu and store NCHW
// with lanes along consecutive pixels (coalesced).
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>

#include "common.h"
#include "tc_common.cuh"
#include "tc_conv_plan.h"
#include "tc_host.h"

namespace onnxb {

namespace {

using namespace tc;

constexpr int kThreads = 352;              // 11 warps
constexpr int kXformWarps = 8;
constexpr int kXformThreads = kXformWarps * 32;
constexpr int kMaxBStages = 6;
constexpr int kSmemLimit = 232448;
constexpr int kBarBytes = 512;
constexpr int kSegBytes = 256;             // >= sizeof(TcConvSegs)
static_assert(sizeof(TcConvSegs) <= kSegBytes, "segment table does not fit its slot");

struct Bars {
    uint64_t raw_full[2], raw_empty[2], a_full[2], a_empty[2];
    uint64_t b_full[kMaxBStages], b_empty[kMaxBStages];
    uint64_t acc_full, acc_empty;
    uint32_t tmem_holder;
};
static_assert(sizeof(Bars) <= kBarBytes, "barrier block too large");

__device__ __forceinline__ float round_tf32(float x) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}

// ------------------------------------------------------------------ weight packing
// Packed layout: [group][channel tile][channel block][tap][chunk of 4 channels][row BN][4],
// i.e. for each (channel block, tap) the exact shared-memory image of the K-major operand:
// 16-byte chunks of 4 consecutive input channels, rows 16 bytes apart.  Values are rounded
// to TF32 (nearest); rows past the group's channels and channels past Cg are zero.
__global__ void pack_weights_kernel(const TcConvPlan g, const float *__restrict__ W, float4 *__restrict__ out) {
    const long long total = g.packed_floats / 4;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long t = i;
        const int row = (int)(t % g.BN); t /= g.BN;
        const int chunk = (int)(t % (kConvKB / 4)); t /= (kConvKB / 4);
        const int tap = (int)(t % g.taps); t /= g.taps;
        const int cb = (int)(t % g.ncb); t /= g.ncb;
        const int ct = (int)(t % g.ctiles); t /= g.ctiles;
        const int grp = (int)t;
        const int mg = ct * g.BN + row;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (mg < g.Mg) {
            const int m = grp * g.Mg + mg;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = cb * kConvKB + chunk * 4 + e;
                if (c < g.Cg) v[e] = round_tf32(__ldg(W + ((size_t)m * g.Cg + c) * g.taps + tap));
            }
        }
        out[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

// ------------------------------------------------------------------ main kernel
__global__ void __launch_bounds__(kThreads, 1)
tc_conv_kernel(const __grid_constant__ CUtensorMap tmX, const TcConvPlan g, const float *__restrict__ X,
               const float *__restrict__ Wpk, const float *__restrict__ bias, float *__restrict__ Y,
               unsigned int *err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_st = smem;
    uint8_t *raw_st = a_st + 2 * (size_t)g.a_stage_bytes;
    uint8_t *b_st = raw_st + 2 * (size_t)g.raw_stage_bytes;
    uint8_t *seg_st = b_st + (size_t)g.nb_stages * g.b_stage_bytes;
    Bars *bars = reinterpret_cast<Bars *>(seg_st + 2 * kSegBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile_rows = g.MT * 128;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->raw_full[s], 1);
            mbar_init(&bars->raw_empty[s], kXformWarps);
            mbar_init(&bars->a_full[s], kXformWarps);
            mbar_init(&bars->a_empty[s], 1);
        }
        for (int s = 0; s < g.nb_stages; ++s) {
            mbar_init(&bars->b_full[s], 1);
            mbar_init(&bars->b_empty[s], 1);
        }
        mbar_init(&bars->acc_full, 1);
        mbar_init(&bars->acc_empty, kXformWarps);
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

    if (warp == 0) {
        // ------------------------------------------------------------ raw activation producer
        if (elect_one()) {
            int rs = 0;
            uint32_t rphase = 0;
            for (long long t = blockIdx.x; t < g.total_tiles; t += gridDim.x) {
                const int ct_all = (int)(t % (g.ctiles * g.group));
                const int grp = ct_all / g.ctiles;
                const long long G0 = (t / (g.ctiles * g.group)) * tile_rows;
                for (int cb = 0; cb < g.ncb; ++cb) {
                    mbar_wait(&bars->raw_empty[rs], rphase ^ 1, err, 11);
                    TcConvSegs *segs = reinterpret_cast<TcConvSegs *>(seg_st + rs * kSegBytes);
                    tc_conv_segments(g, G0, *segs);
                    float *dst = reinterpret_cast<float *>(raw_st + (size_t)rs * g.raw_stage_bytes);
                    const int c0 = grp * g.Cg + cb * kConvKB;
                    if (g.raw_mode == 0) {
                        mbar_arrive_expect_tx(&bars->raw_full[rs], (uint32_t)segs->total_floats * 4u);
                        for (int i = 0; i < segs->nseg; ++i) {
                            const int plane0 = (segs->n_first + i) * g.C + c0;
                            for (int j = 0; j < segs->nbox[i]; ++j)
                                tma_load_2d(dst + segs->base[i] + j * (kConvKB * g.BOXP), &tmX, &bars->raw_full[rs],
                                            segs->f0[i] + j * g.BOXP, plane0);
                        }
                    } else {
                        // whole-image slabs [channel][H*W]; clip at the end of X
                        const long long HW = (long long)g.H * g.W;
                        const long long planes_total = (long long)g.N * g.C;
                        uint32_t bytes[kConvMaxSeg];
                        uint32_t total = 0;
                        for (int i = 0; i < segs->nseg; ++i) {
                            bytes[i] = 0;
                            if (segs->nbox[i]) {
                                const long long plane0 = (long long)(segs->n_first + i) * g.C + c0;
                                long long nch = planes_total - plane0;
                                if (nch > kConvKB) nch = kConvKB;
                                bytes[i] = nch > 0 ? (uint32_t)(nch * HW * 4) : 0u;
                                total += bytes[i];
                            }
                        }
                        mbar_arrive_expect_tx(&bars->raw_full[rs], total);
                        for (int i = 0; i < segs->nseg; ++i)
                            if (bytes[i])
                                bulk_load_1d(dst + segs->base[i],
                                             X + ((long long)(segs->n_first + i) * g.C + c0) * HW, bytes[i],
                                             &bars->raw_full[rs]);
                    }
                    if (++rs == 2) { rs = 0; rphase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ weight producer
        if (elect_one()) {
            int bs = 0;
            uint32_t bphase = 0;
            const long long per_ct = (long long)g.ncb * g.taps * g.BN * kConvKB;   // floats per channel tile
            for (long long t = blockIdx.x; t < g.total_tiles; t += gridDim.x) {
                const int ct_all = (int)(t % (g.ctiles * g.group));
                const float *src = Wpk + ct_all * per_ct;
                for (int step = 0; step < g.ncb * g.taps; ++step) {
                    mbar_wait(&bars->b_empty[bs], bphase ^ 1, err, 12);
                    mbar_arrive_expect_tx(&bars->b_full[bs], (uint32_t)g.b_stage_bytes);
                    bulk_load_1d(b_st + (size_t)bs * g.b_stage_bytes, src + (long long)step * g.BN * kConvKB,
                                 (uint32_t)g.b_stage_bytes, &bars->b_full[bs]);
                    if (++bs == g.nb_stages) { bs = 0; bphase ^= 1; }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            int as = 0, bs = 0;
            uint32_t aphase = 0, bphase = 0, accphase = 0;
            for (long long t = blockIdx.x; t < g.total_tiles; t += gridDim.x) {
                mbar_wait(&bars->acc_empty, accphase ^ 1, err, 13);
                tc_fence_after_sync();
                uint32_t accumulate = 0;
                for (int cb = 0; cb < g.ncb; ++cb) {
                    mbar_wait(&bars->a_full[as], aphase, err, 14);
                    const uint32_t a_base = smem_u32(a_st + (size_t)as * g.a_stage_bytes);
                    for (int tap = 0; tap < g.taps; ++tap) {
                        mbar_wait(&bars->b_full[bs], bphase, err, 15);
                        tc_fence_after_sync();
                        const uint32_t b_base = smem_u32(b_st + (size_t)bs * g.b_stage_bytes);
                        const uint32_t a_tap = a_base + (uint32_t)g.tap_plane[tap] * g.plane_pitch +
                                               (uint32_t)g.tap_shift[tap] * 16u;
#pragma unroll
                        for (int j = 0; j < kConvKB / 8; ++j) {
                            // no-swizzle K-major operands: rows 16 bytes apart (8-row groups 128 bytes
                            // apart), the two 16-byte K chunks of one instruction one chunk pitch apart
                            const uint64_t bd = make_smem_desc(b_base + (uint32_t)(2 * j) * g.BN * 16u,
                                                               (uint32_t)g.BN * 16u, 128, kSwizzleNone);
                            for (int mt = 0; mt < g.MT; ++mt) {
                                const uint64_t ad =
                                    make_smem_desc(a_tap + (uint32_t)(2 * j) * g.chunk_pitch + (uint32_t)mt * 2048u,
                                                   (uint32_t)g.chunk_pitch, 128, kSwizzleNone);
                                mma_tf32(tmem_base + (uint32_t)mt * 256u, ad, bd, g.idesc, accumulate);
                            }
                            accumulate = 1;
                        }
                        mma_commit(&bars->b_empty[bs]);
                        if (++bs == g.nb_stages) { bs = 0; bphase ^= 1; }
                    }
                    mma_commit(&bars->a_empty[as]);
                    if (++as == 2) { as = 0; aphase ^= 1; }
                }
                mma_commit(&bars->acc_full);
                accphase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------ transform + epilogue warps
        const int xw = warp - 3;                   // 0..7
        const int xt = xw * 32 + lane;             // 0..255
        const int quarter = warp & 3;              // TMEM lane quarter this warp may read
        const int hf = xw >> 2;
        const int cp = g.raw_mode == 1 ? g.H * g.W : g.BOXP;    // channel pitch inside the raw stage
        const int per_stage_slots = g.planes * g.SLOTS;
        const long long PQ = (long long)g.P * g.Q;
        int rs = 0, as = 0;
        uint32_t rphase = 0, aphase = 0, accphase = 0;
        for (long long t = blockIdx.x; t < g.total_tiles; t += gridDim.x) {
            const int ct_all = (int)(t % (g.ctiles * g.group));
            const int grp = ct_all / g.ctiles, ct = ct_all % g.ctiles;
            const long long G0 = (t / (g.ctiles * g.group)) * tile_rows;
            int off[4];                            // raw float offset of channel 0 for up to 4 owned slots
            for (int cb = 0; cb < g.ncb; ++cb) {
                mbar_wait(&bars->raw_full[rs], rphase, err, 16);
                if (cb == 0) {
                    const TcConvSegs *segs = reinterpret_cast<const TcConvSegs *>(seg_st + rs * kSegBytes);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        off[i] = -1;
                        const int idx = xt + i * kXformThreads;
                        if (idx < per_stage_slots) {
                            const int pl = idx / g.SLOTS, j = idx - pl * g.SLOTS;
                            const long long Gs = G0 + j;
                            if (Gs < g.total_slots) {
                                const int n = (int)(Gs / g.L);
                                const int u = (int)(Gs - (long long)n * g.L);
                                const int hq = u / g.Ws, wq = u - hq * g.Ws;
                                const int h = hq * g.sh + g.pa[pl] - g.pt;
                                const int w = wq * g.sw + g.pb[pl] - g.pl;
                                const int sg = n - segs->n_first;
                                if ((unsigned)h < (unsigned)g.H && (unsigned)w < (unsigned)g.W && sg < segs->nseg) {
                                    const int f = h * g.W + w - segs->f0[sg];
                                    if (g.raw_mode == 1) off[i] = segs->base[sg] + f;
                                    else {
                                        const int bx = f / g.BOXP;
                                        off[i] = segs->base[sg] + bx * (kConvKB * g.BOXP) + (f - bx * g.BOXP);
                                    }
                                }
                            }
                        }
                    }
                }
                mbar_wait(&bars->a_empty[as], aphase ^ 1, err, 17);
                const float *raw = reinterpret_cast<const float *>(raw_st + (size_t)rs * g.raw_stage_bytes);
                uint8_t *adst = a_st + (size_t)as * g.a_stage_bytes;
                const int c_left = g.Cg - cb * kConvKB;    // channels of this block that exist
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int idx = xt + i * kXformThreads;
                    if (idx < per_stage_slots) {
#pragma unroll
                        for (int ch = 0; ch < kConvKB / 4; ++ch) {
                            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (off[i] >= 0) {
                                const float *r = raw + off[i] + (ch * 4) * cp;
                                const int left = c_left - ch * 4;
                                if (left > 0) v.x = round_tf32(r[0]);
                                if (left > 1) v.y = round_tf32(r[cp]);
                                if (left > 2) v.z = round_tf32(r[2 * cp]);
                                if (left > 3) v.w = round_tf32(r[3 * cp]);
                            }
                            *reinterpret_cast<float4 *>(adst + (size_t)ch * g.chunk_pitch + (size_t)idx * 16) = v;
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&bars->a_full[as]);
                    mbar_arrive(&bars->raw_empty[rs]);
                }
                if (++rs == 2) { rs = 0; rphase ^= 1; }
                if (++as == 2) { as = 0; aphase ^= 1; }
            }

            // ---- epilogue of this tile
            mbar_wait(&bars->acc_full, accphase, err, 18);
            tc_fence_after_sync();
            const int nch = (g.BN + 31) / 32;
            int mt, ch_lo, ch_hi;
            if (g.MT == 2) { mt = hf; ch_lo = 0; ch_hi = nch; }
            else { mt = 0; ch_lo = hf ? (nch + 1) / 2 : 0; ch_hi = hf ? nch : (nch + 1) / 2; }
            const long long G = G0 + mt * 128 + quarter * 32 + lane;
            bool valid = G < g.total_slots;
            long long ybase = 0;
            if (valid) {
                const int n = (int)(G / g.L);
                const int u = (int)(G - (long long)n * g.L);
                const int p = u / g.Ws, q = u - p * g.Ws;
                valid = p < g.P && q < g.Q;
                ybase = ((long long)n * g.M * g.P + p) * g.Q + q;
            }
            for (int chunk = ch_lo; chunk < ch_hi; ++chunk) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * 256 + chunk * 32), v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int mg = ct * g.BN + chunk * 32 + j;     // channel within the group (warp-uniform)
                    if (mg < g.Mg && chunk * 32 + j < g.BN) {
                        const int m = grp * g.Mg + mg;
                        float x = __uint_as_float(v[j]) + (bias ? __ldg(bias + m) : 0.f);
                        if (g.relu) x = x > 0.f ? x : 0.f;
                        if (valid) Y[ybase + (long long)m * PQ] = x;
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_empty);
            accphase ^= 1;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
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

bool fill_plan(const ConvGeom &c, int MT, int BN, TcConvPlan &g) {
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
    g.planes = 0;
    for (int i = 0; i < ah.npar; ++i)
        for (int j = 0; j < aw.npar; ++j) { g.pa[g.planes] = ah.par[i]; g.pb[g.planes] = aw.par[j]; ++g.planes; }
    g.a_min = ah.par[0]; g.a_max = ah.par[ah.npar - 1];
    for (int r = 0; r < c.kH; ++r)
        for (int s = 0; s < c.kW; ++s) {
            const int a = (r * c.dh) % c.sh, b = (s * c.dw) % c.sw;
            int pl = 0;
            while (g.pa[pl] != a || g.pb[pl] != b) ++pl;
            g.tap_plane[r * c.kW + s] = pl;
            g.tap_shift[r * c.kW + s] = ((r * c.dh) / c.sh) * g.Ws + (s * c.dw) / c.sw;
        }
    const long long maxshift = (long long)ah.Amax * g.Ws + aw.Amax;
    g.MT = MT; g.BN = BN;
    g.ctiles = (c.Mg + BN - 1) / BN;
    const long long slots = (long long)MT * 128 + maxshift;
    if (slots * g.planes > 4 * kXformThreads) return false;      // each transform thread owns at most 4 slots
    g.SLOTS = (int)slots;
    if ((g.SLOTS + L - 2) / L + 1 > kConvMaxSeg) return false;
    g.ncb = (c.Cg + kConvKB - 1) / kConvKB;
    const long long ptiles = (g.total_slots + MT * 128 - 1) / (MT * 128);
    if (ptiles > 0x7fffffffLL) return false;
    g.pix_tiles = (int)ptiles;
    g.total_tiles = ptiles * g.ctiles * c.group;
    // raw staging mode
    const long long HW = (long long)c.H * c.W;
    if (HW % 4 == 0) {
        g.raw_mode = 0;
    } else if (c.Cg % 4 == 0 && c.C % 4 == 0 && HW * kConvKB * 4 <= 32768) {
        g.raw_mode = 1;
    } else {
        return false;
    }
    g.plane_pitch = g.SLOTS * 16;
    g.chunk_pitch = g.planes * g.plane_pitch;
    if (g.chunk_pitch >= (1 << 18)) return false;
    g.a_stage_bytes = (kConvKB / 4) * g.chunk_pitch;
    g.a_stage_bytes = (g.a_stage_bytes + 127) / 128 * 128;
    g.b_stage_bytes = BN * kConvKB * 4;
    g.idesc = tc::make_idesc_tf32(128, BN, 0, 0);
    g.packed_floats = (long long)c.group * g.ctiles * g.ncb * g.taps * BN * kConvKB;
    // raw stage size: widest flat pixel range any tile needs, found by walking the tiles
    g.BOXP = 256;
    if (g.raw_mode == 0) {
        int widest = 4;
        const long long walk = std::min<long long>(ptiles, L + 2);
        for (long long i = 0; i <= walk; ++i) {
            const long long pt = i < walk ? i : ptiles - 1;
            const long long G0 = pt * MT * 128;
            long long Gend = std::min<long long>(G0 + g.SLOTS, g.total_slots);
            const int n_first = (int)(G0 / L), n_last = (int)((Gend - 1) / L);
            for (int n = n_first; n <= n_last; ++n) {
                const long long lo = std::max<long long>(G0, (long long)n * L), hi = std::min<long long>(Gend, (long long)(n + 1) * L);
                const int hq_lo = (int)((lo - (long long)n * L) / g.Ws), hq_hi = (int)((hi - 1 - (long long)n * L) / g.Ws);
                int h_min = std::max(0, hq_lo * c.sh + g.a_min - c.pt);
                int h_max = std::min(c.H - 1, hq_hi * c.sh + g.a_max - c.pt);
                if (h_min > h_max) continue;
                const int f0 = (h_min * c.W) & ~3;
                widest = std::max(widest, (h_max + 1) * c.W - f0);
            }
        }
        widest = (widest + 3) / 4 * 4;
        g.BOXP = std::min(256, widest);
    }
    {
        int worst = 0;
        TcConvSegs segs;
        const long long walk = std::min<long long>(ptiles, L + 2);
        for (long long i = 0; i <= walk; ++i) {
            const long long pt = i < walk ? i : ptiles - 1;
            tc_conv_segments(g, pt * MT * 128, segs);
            worst = std::max(worst, segs.total_floats);
        }
        g.raw_stage_bytes = (worst * 4 + 127) / 128 * 128;
        if (g.raw_stage_bytes == 0) g.raw_stage_bytes = 128;
    }
    const long long fixed = 1024 + 2LL * g.a_stage_bytes + 2LL * g.raw_stage_bytes + 2 * kSegBytes + kBarBytes;
    const long long room = kSmemLimit - fixed;
    if (room < 2LL * g.b_stage_bytes) return false;
    g.nb_stages = (int)std::min<long long>(kMaxBStages, room / g.b_stage_bytes);
    return true;
}

}  // namespace

bool tc_conv_plan(const ConvGeom &c, TcConvPlan &plan) {
    if (c.Cg < 16) return false;                  // thin contraction: SIMT family
    const int sms = 148;
    const int bn0 = pick_conv_bn(c.Mg);
    // Candidate tiles, largest first: 256 or 128 pixels x up to 256 channels.  The cost model is
    // waves x (MMA time of one tile, with a floor where narrow tiles become shared-memory bound).
    int cand[5][2];
    int ncand = 0;
    cand[ncand][0] = 2; cand[ncand++][1] = bn0;
    cand[ncand][0] = 1; cand[ncand++][1] = bn0;
    if (bn0 > 128) {
        cand[ncand][0] = 2; cand[ncand++][1] = 128;
        cand[ncand][0] = 1; cand[ncand++][1] = 128;
    }
    if (bn0 > 64) { cand[ncand][0] = 1; cand[ncand++][1] = 64; }
    bool have = false;
    double best_cost = 0;
    for (int i = 0; i < ncand; ++i) {
        TcConvPlan p;
        if (!fill_plan(c, cand[i][0], cand[i][1], p)) continue;
        const long long waves = (p.total_tiles + sms - 1) / sms;
        const double cost = (double)waves * p.MT * std::max(p.BN, 96);
        if (!have || cost < best_cost * 0.999) {
            have = true;
            best_cost = cost;
            plan = p;
        }
    }
    return have;
}

size_t tc_conv_workspace_bytes(const TcConvPlan &plan) { return (size_t)plan.packed_floats * 4; }

int launch_tc_conv(const TcConvPlan &plan, const float *X, const float *W, const float *B, float *Y,
                   void *workspace, void *stream) {
    using namespace tc_host;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned int *err = device_status_ptr();
    if (!err) return (int)cudaErrorUnknown;

    // 1. pack + round the weights into the workspace
    {
        const long long vec = plan.packed_floats / 4;
        const int blocks = (int)std::min<long long>((vec + 255) / 256, 148 * 16);
        pack_weights_kernel<<<blocks, 256, 0, st>>>(plan, W, reinterpret_cast<float4 *>(workspace));
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return (int)e;
    }
    // 2. the convolution
    CUtensorMap tmX;
    if (plan.raw_mode == 0) {
        const uint64_t dims[2] = {(uint64_t)plan.H * plan.W, (uint64_t)plan.N * plan.C};
        const uint64_t str[1] = {(uint64_t)plan.H * plan.W * 4};
        const uint32_t box[2] = {(uint32_t)plan.BOXP, (uint32_t)kConvKB};
        if (!make_tmap(&tmX, X, 2, dims, str, box, kTmapSwizzleNone)) return (int)cudaErrorInvalidValue;
    } else {
        memset(&tmX, 0, sizeof tmX);
    }
    const size_t smem = 1024 + 2 * (size_t)plan.a_stage_bytes + 2 * (size_t)plan.raw_stage_bytes +
                        (size_t)plan.nb_stages * plan.b_stage_bytes + 2 * kSegBytes + kBarBytes;
    cudaError_t e = cudaFuncSetAttribute(tc_conv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return (int)e;
    const int sms = num_sms();
    const int grid = (int)std::min<long long>(plan.total_tiles, sms);
    tc_conv_kernel<<<grid, kThreads, smem, st>>>(tmX, plan, X, reinterpret_cast<const float *>(workspace), B, Y, err);
    count_launch();
    return (int)cudaGetLastError();
}

}  // namespace onnxb
