// Geometry of the implicit-GEMM convolution kernel, shared by host planning and
// device code (plain integer arithmetic, no CUDA types).
//
// "Slot space".  For every image the kernel lays the (zero-padded, stride-decimated)
// input out as a grid of Hs x Ws slots per parity plane; slot (hq, wq) of plane (a, b)
// holds the padded input pixel (hq*sh + a, wq*sw + b).  Output pixel (p, q) is anchored
// at slot u = p*Ws + q, and filter tap (r, s) reads plane ((r*dh) % sh, (s*dw) % sw) at
// slot u + ((r*dh)/sh)*Ws + (s*dw)/sw: a fixed shift per tap.  Images follow each other
// every L = Hs*Ws slots, so a GEMM row tile is simply 128 consecutive global slots, and
// the im2col operand of a tap is the same shared-memory tile read from a shifted start
// address.  Hs and Ws are chosen as small as possible: the trailing zero padding of one
// row (image) is allowed to alias the leading zero padding of the next.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define ONNXB_HD __host__ __device__
#else
#define ONNXB_HD
#endif

namespace onnxb {

constexpr int kConvMaxPlanes = 4;
constexpr int kConvMaxTaps = 64;
constexpr int kConvMaxSteps = 128;     // MMA K-steps (8 reduction terms each) per channel block
constexpr int kConvMaxSeg = 8;

struct ConvDivisor {
    uint32_t d, m, s1, s2;
};

struct TcConvPlan {
    // problem
    int N, C, H, W, M, Cg, Mg, kH, kW, P, Q, pt, pl, sh, sw, dh, dw, group, relu;
    // slot space
    int Hs, Ws, L;
    long long total_slots;           // N * L
    int planes, pa[kConvMaxPlanes], pb[kConvMaxPlanes];
    int a_min, a_max;                // smallest / largest used row parity
    int taps;
    // Reduction blocking.  A channel block holds KB input channels as KB/4 chunks of 4 (one 16-byte
    // operand row per slot and chunk).  One MMA K-step consumes two chunks:
    //   KB = 16 ("channel pairs"): chunks 2j, 2j+1 of the same tap, two steps per tap;
    //   KB = 4  ("tap pairs", for C/group < 16): the single chunk read at two taps of the same plane.
    int KB, nchunks, n_steps;
    uint32_t step_a[kConvMaxSteps];      // A descriptor low word relative to the stage: offset/16 | (LBO/16) << 16
    short src_tap[kConvMaxSteps][2];     // which filter tap feeds chunk 0 / 1 of the step's weights (-1: zeros)
    short src_c0[kConvMaxSteps][2];      // and from which channel offset inside the block
    // tiling
    int ctas;                        // CTAs working on one tile: 1, or 2 (a cluster pair issuing M = 256 MMAs)
    int MT;                          // 128-row accumulator tiles per CTA (1 or 2)
    int BN, ctiles;                  // output channels per tile, tiles per group
    int BNH;                         // weight rows each CTA stages per K-step = BN / ctas
    int SLOTS;                       // slots per plane held in one A stage = MT*128 + largest tap shift
    int ncb;                         // channel blocks = ceil(Cg / KB)
    int pix_tiles;                   // ceil(total_slots / (ctas*MT*128))
    long long total_tiles;
    // raw staging
    int raw_mode;                    // 0: tensor-map boxes [KB][BOXP] over X seen as (H*W, N*C); 1: whole-image slabs
    int BOXP;
    // shared memory carve-up (bytes)
    int a_stage_bytes, raw_stage_bytes, b_stage_bytes, nb_stages, nr_stages, na_stages;
    int spb, b_step_bytes, b_steps;  // K-steps per weight stage, bytes of one step's weights, weight stages per block
    int chunk_pitch, plane_pitch;    // bytes between 4-channel chunks / parity planes inside an A stage
    uint32_t idesc;
    long long packed_floats;         // size of the packed weight buffer
    // divisors device code needs per slot, as multiply-and-shift constants (see conv_fdiv)
    ConvDivisor dv_L, dv_Ws, dv_Hs, dv_BOXP, dv_SLOTS, dv_pss;
    int boxp_shift;                  // log2(BOXP) when BOXP is a power of two, else -1
    int epi_warps;                   // epilogue warps of the launch: 8, or 4 (then 128 registers per thread)
    int relay;                       // pairs: the odd CTA's "operand stage written" goes through its relay warp
};

// floor(n / d) for any 32-bit unsigned n.  On the device: the round-up multiply-and-shift method
// (Granlund and Montgomery, "Division by invariant integers using multiplication"): with
// l = ceil(log2 d) and m = floor(2^32 (2^l - d) / d) + 1, t = high32(m * n) and
// q = (t + ((n - t) >> min(l, 1))) >> max(l - 1, 0).  On the host: plain division.
// (The host passes the divisor itself: while a plan is being filled its constants are not yet set.)
ONNXB_HD inline int conv_fdiv(int n, int d, const ConvDivisor &dv) {
#if defined(__CUDA_ARCH__)
    (void)d;
    const uint32_t un = (uint32_t)n, t = __umulhi(dv.m, un);
    return (int)((t + ((un - t) >> dv.s1)) >> dv.s2);
#else
    (void)dv;
    return (int)((uint32_t)n / (uint32_t)d);
#endif
}
inline ConvDivisor conv_divisor(int d) {
    ConvDivisor dv;
    dv.d = (uint32_t)d;
    int l = 0;
    while ((1ull << l) < (unsigned long long)d) ++l;
    dv.m = (uint32_t)(((1ull << 32) * ((1ull << l) - (unsigned long long)d)) / (unsigned long long)d + 1);
    dv.s1 = l < 1 ? (uint32_t)l : 1u;
    dv.s2 = l > 1 ? (uint32_t)(l - 1) : 0u;
    return dv;
}

struct TcConvSegs {
    int n_first, nseg;
    int hq0, wq0;                    // slot row / column of the tile's first slot within image n_first
    int f0[kConvMaxSeg];             // first flat pixel (h*W + w) staged for the image
    int base[kConvMaxSeg];           // float offset of the image's data inside the raw stage
    int nbox[kConvMaxSeg];           // boxes (mode 0) / 1 (mode 1) / 0 when nothing of the image is needed
    int total_floats;
};

// Which part of which images the A stage of the tile starting at global slot G0 needs.
ONNXB_HD inline void tc_conv_segments(const TcConvPlan &g, long long G0, TcConvSegs &t) {
    long long Gend = G0 + g.SLOTS;
    if (Gend > g.total_slots) Gend = g.total_slots;
    if (G0 >= g.total_slots) {       // the second CTA of a pair on the last, half-empty tile
        t.n_first = g.N;
        t.nseg = 0;
        t.hq0 = t.wq0 = 0;
        t.total_floats = 0;
        return;
    }
    t.n_first = conv_fdiv((int)G0, g.L, g.dv_L);
    {
        const int u0 = (int)(G0 - (long long)t.n_first * g.L);
        t.hq0 = conv_fdiv(u0, g.Ws, g.dv_Ws);
        t.wq0 = u0 - t.hq0 * g.Ws;
    }
    const int n_last = conv_fdiv((int)(Gend - 1), g.L, g.dv_L);
    t.nseg = n_last - t.n_first + 1;
    if (t.nseg > kConvMaxSeg) t.nseg = kConvMaxSeg;   // excluded by the planner
    int base = 0;
    for (int i = 0; i < t.nseg; ++i) {
        const long long n = t.n_first + i;
        const long long lo = G0 > n * g.L ? G0 : n * g.L;
        const long long hi = Gend < (n + 1) * g.L ? Gend : (n + 1) * g.L;
        const int u_lo = (int)(lo - n * g.L), u_hi = (int)(hi - n * g.L);   // [u_lo, u_hi)
        const int hq_lo = conv_fdiv(u_lo, g.Ws, g.dv_Ws), hq_hi = conv_fdiv(u_hi - 1, g.Ws, g.dv_Ws);
        int h_min = hq_lo * g.sh + g.a_min - g.pt;
        int h_max = hq_hi * g.sh + g.a_max - g.pt;
        if (h_min < 0) h_min = 0;
        if (h_max > g.H - 1) h_max = g.H - 1;
        t.base[i] = base;
        if (h_min > h_max) {
            t.f0[i] = 0;
            t.nbox[i] = 0;
        } else if (g.raw_mode == 1) {
            t.f0[i] = 0;
            t.nbox[i] = 1;
            base += g.KB * g.H * g.W;
        } else {
            const int f0 = (h_min * g.W) & ~3;
            const int len = (h_max + 1) * g.W - f0;
            t.f0[i] = f0;
            t.nbox[i] = conv_fdiv(len + g.BOXP - 1, g.BOXP, g.dv_BOXP);
            base += t.nbox[i] * g.BOXP * g.KB;
        }
    }
    t.total_floats = base;
}

}  // namespace onnxb
