// Descriptor layer: ONNX Conv attribute validation, auto_pad resolution, output
// shape inference (the shape-inference pass of Sec. 3.4.2 restricted to one
// operator with static shapes) and kernel choice.  Host only; no CUDA call.
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.h"

namespace onnxb {

std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_override{-2};   // -2 = environment not read yet

int kernel_override() {
    int v = g_override.load(std::memory_order_acquire);
    if (v == -2) {
        v = -1;
        if (const char *e = std::getenv("ONNXB_FORCE")) {
            if (!std::strcmp(e, "simt")) v = ONNXB_KERNEL_SIMT_DIRECT;
            else if (!std::strcmp(e, "mma")) v = ONNXB_KERNEL_MMA_IMPLICIT;
        }
        int expected = -2;
        g_override.compare_exchange_strong(expected, v);
        v = g_override.load(std::memory_order_acquire);
    }
    return v;
}

static const int64_t kMaxElems = 2147483647LL;

static bool mul_fits(int64_t a, int64_t b, int64_t c, int64_t d) {
    // all factors are >= 1 here
    __int128 t = (__int128)a * b;
    t *= c;
    t *= d;
    return t <= (__int128)kMaxElems;
}

}  // namespace onnxb

using namespace onnxb;

extern "C" onnxb_status onnx_conv2d_desc(const onnxb_conv2d_attrs *a, onnxb_conv2d_desc_t *out) {
    if (!a || !out) return ONNXB_ERR_NULL;
    *out = nullptr;
    if (a->reserved != 0) return ONNXB_ERR_ATTR;

    const int64_t N = a->x_dims[0], C = a->x_dims[1], H = a->x_dims[2], W = a->x_dims[3];
    const int64_t M = a->w_dims[0], Cg = a->w_dims[1], kH = a->w_dims[2], kW = a->w_dims[3];
    if (N < 1 || C < 1 || H < 1 || W < 1 || M < 1 || Cg < 1 || kH < 1 || kW < 1) return ONNXB_ERR_SHAPE;

    // kernel_shape: absent (0,0) means "take it from W"
    if (a->kernel_shape[0] != 0 || a->kernel_shape[1] != 0) {
        if (a->kernel_shape[0] != kH || a->kernel_shape[1] != kW) return ONNXB_ERR_ATTR;
    }

    int64_t st[2], di[2];
    for (int i = 0; i < 2; ++i) {
        st[i] = a->strides[i];
        di[i] = a->dilations[i];
    }
    if (st[0] == 0 && st[1] == 0) st[0] = st[1] = 1;
    if (di[0] == 0 && di[1] == 0) di[0] = di[1] = 1;
    if (st[0] < 1 || st[1] < 1 || di[0] < 1 || di[1] < 1) return ONNXB_ERR_ATTR;

    int64_t group = a->group == 0 ? 1 : a->group;
    if (group < 1) return ONNXB_ERR_ATTR;
    if (C % group != 0 || M % group != 0 || Cg != C / group) return ONNXB_ERR_SHAPE;

    int64_t pads[4] = {a->pads[0], a->pads[1], a->pads[2], a->pads[3]};
    for (int i = 0; i < 4; ++i)
        if (pads[i] < 0) return ONNXB_ERR_UNSUPPORTED;

    const int64_t in[2] = {H, W};
    const int64_t eff[2] = {(kH - 1) * di[0] + 1, (kW - 1) * di[1] + 1};
    switch (a->auto_pad) {
        case ONNXB_NOTSET:
            break;
        case ONNXB_VALID:
        case ONNXB_SAME_UPPER:
        case ONNXB_SAME_LOWER:
            if (pads[0] || pads[1] || pads[2] || pads[3]) return ONNXB_ERR_ATTR;
            if (a->auto_pad != ONNXB_VALID) {
                for (int ax = 0; ax < 2; ++ax) {
                    const int64_t o = (in[ax] + st[ax] - 1) / st[ax];
                    int64_t total = (o - 1) * st[ax] + eff[ax] - in[ax];
                    if (total < 0) total = 0;
                    const int64_t lo = total / 2, hi = total - lo;
                    pads[ax] = a->auto_pad == ONNXB_SAME_UPPER ? lo : hi;
                    pads[ax + 2] = a->auto_pad == ONNXB_SAME_UPPER ? hi : lo;
                }
            }
            break;
        default:
            return ONNXB_ERR_ATTR;
    }

    int64_t outdim[2];
    for (int ax = 0; ax < 2; ++ax) {
        const int64_t num = in[ax] + pads[ax] + pads[ax + 2] - eff[ax];
        if (num < 0) return ONNXB_ERR_SHAPE;
        outdim[ax] = num / st[ax] + 1;
    }
    const int64_t P = outdim[0], Q = outdim[1];

    if (!mul_fits(N, C, H, W) || !mul_fits(M, Cg, kH, kW) || !mul_fits(N, M, P, Q)) return ONNXB_ERR_UNSUPPORTED;
    // padded coordinates are formed in 32-bit arithmetic on the device
    for (int ax = 0; ax < 2; ++ax) {
        if (pads[ax] > (1 << 20) || pads[ax + 2] > (1 << 20) || st[ax] > (1 << 20) || di[ax] > (1 << 20))
            return ONNXB_ERR_UNSUPPORTED;
        if ((outdim[ax] - 1) * st[ax] + eff[ax] > kMaxElems) return ONNXB_ERR_UNSUPPORTED;
    }

    onnxb_conv2d_desc_s *d = new (std::nothrow) onnxb_conv2d_desc_s();
    if (!d) return ONNXB_ERR_CUDA;
    ConvGeom &g = d->g;
    g.N = (int)N; g.C = (int)C; g.H = (int)H; g.W = (int)W;
    g.M = (int)M; g.Cg = (int)Cg; g.kH = (int)kH; g.kW = (int)kW;
    g.P = (int)P; g.Q = (int)Q;
    g.pt = (int)pads[0]; g.pl = (int)pads[1]; g.pb = (int)pads[2]; g.pr = (int)pads[3];
    g.sh = (int)st[0]; g.sw = (int)st[1]; g.dh = (int)di[0]; g.dw = (int)di[1];
    g.group = (int)group; g.Mg = (int)(M / group);
    g.has_bias = a->has_bias != 0; g.relu = a->fuse_relu != 0;
    d->y_dims[0] = N; d->y_dims[1] = M; d->y_dims[2] = P; d->y_dims[3] = Q;
    for (int i = 0; i < 4; ++i) d->pads[i] = pads[i];

    // Dispatch (tailoring the code to the problem at hand): depthwise and thin
    // contractions run on the SIMT family.
    const int forced = kernel_override();
    int family = ONNXB_KERNEL_SIMT_DIRECT;
    if (simt_depthwise_supports(g)) family = ONNXB_KERNEL_SIMT_DEPTHWISE;
    else if (conv_fits_mma_gemm(g)) family = ONNXB_KERNEL_MMA_GEMM;
    else if (conv_fits_mma_gather_gemm(g)) family = ONNXB_KERNEL_MMA_GATHER_GEMM;
    else if (tc_conv_plan(g, d->plan)) family = ONNXB_KERNEL_MMA_IMPLICIT;
    if (forced == ONNXB_KERNEL_SIMT_DIRECT) family = ONNXB_KERNEL_SIMT_DIRECT;
    else if (forced == ONNXB_KERNEL_SIMT_DEPTHWISE) {
        if (!simt_depthwise_supports(g)) { delete d; return ONNXB_ERR_UNSUPPORTED; }
        family = ONNXB_KERNEL_SIMT_DEPTHWISE;
    } else if (forced == ONNXB_KERNEL_MMA_GEMM) {
        if (!conv_fits_mma_gemm(g)) { delete d; return ONNXB_ERR_UNSUPPORTED; }
        family = ONNXB_KERNEL_MMA_GEMM;
    } else if (forced == ONNXB_KERNEL_MMA_GATHER_GEMM) {
        if (!conv_fits_mma_gather_gemm(g)) { delete d; return ONNXB_ERR_UNSUPPORTED; }
        family = ONNXB_KERNEL_MMA_GATHER_GEMM;
    } else if (forced == ONNXB_KERNEL_MMA_IMPLICIT) {
        if (!tc_conv_plan(g, d->plan, true)) { delete d; return ONNXB_ERR_UNSUPPORTED; }
        family = ONNXB_KERNEL_MMA_IMPLICIT;
    }
    d->family = family;
    d->workspace_bytes = family == ONNXB_KERNEL_MMA_IMPLICIT     ? tc_conv_workspace_bytes(d->plan)
                         : family == ONNXB_KERNEL_MMA_GATHER_GEMM ? conv_gather_workspace_bytes(g) + (size_t)g.M * g.C * 4
                         : family == ONNXB_KERNEL_MMA_GEMM        ? (size_t)g.M * g.C * 4      // W rounded to TF32
                                                                  : 0;
    *out = d;
    return ONNXB_OK;
}

extern "C" onnxb_status onnx_conv2d_desc_query(onnxb_conv2d_desc_t d, int64_t y_dims[4],
                                               int64_t resolved_pads[4], size_t *workspace_bytes) {
    if (!d) return ONNXB_ERR_NULL;
    if (y_dims) std::memcpy(y_dims, d->y_dims, sizeof d->y_dims);
    if (resolved_pads) std::memcpy(resolved_pads, d->pads, sizeof d->pads);
    if (workspace_bytes) *workspace_bytes = d->workspace_bytes;
    return ONNXB_OK;
}

extern "C" int onnx_conv2d_desc_query_kernel(onnxb_conv2d_desc_t d) { return d ? d->family : -1; }

extern "C" void onnx_conv2d_desc_destroy(onnxb_conv2d_desc_t d) { delete d; }

extern "C" void onnxb_set_kernel_override(int family) {
    kernel_override();   // make sure the environment has been consumed first
    g_override.store(family < 0 ? -1 : family, std::memory_order_release);
}

extern "C" uint64_t onnxb_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" const char *onnxb_status_string(onnxb_status s) {
    switch (s) {
        case ONNXB_OK: return "ok";
        case ONNXB_ERR_NULL: return "null pointer";
        case ONNXB_ERR_ATTR: return "invalid attribute";
        case ONNXB_ERR_SHAPE: return "inconsistent shape";
        case ONNXB_ERR_UNSUPPORTED: return "unsupported";
        case ONNXB_ERR_WORKSPACE: return "workspace too small";
        case ONNXB_ERR_CUDA: return "CUDA error";
        case ONNXB_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}
