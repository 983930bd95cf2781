"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI,
run the oracle on the same seeded inputs, compare element by element."""
import numpy as np

import oracle

# |gpu - oracle| <= REL * sum|x*w| + ABS per output element.  The relative part
# covers TF32 operand rounding (2^-11 per operand, 2 operands: 9.8e-4 per term
# at most) and fp32 accumulation; the absolute part covers the single fp32
# rounding of the bias / beta*C addition and of the stored result.
REL, ABS = 1e-3, 1e-5


def worst_ratio(got, want, S):
    """max over elements of |got - want| / (REL*S + ABS); parity holds iff <= 1."""
    got = np.asarray(got, dtype=np.float64)
    if got.shape != want.shape:
        raise AssertionError(f"shape {got.shape} != {want.shape}")
    if got.size == 0:
        return 0.0
    if not np.isfinite(got).all():
        return float("inf")
    return float(np.max(np.abs(got - want) / (REL * S + ABS)))


def conv_case_kwargs(case):
    return dict(pads=case.pads, strides=case.strides, dilations=case.dilations, group=case.group)


def run_conv_gpu(binding, torch, X, W, B, *, pads=(0, 0, 0, 0), strides=(1, 1), dilations=(1, 1), group=1,
                 relu=False, auto_pad="NOTSET", canary=True):
    """Returns (Y as numpy, kernel family).  With canary, Y sits between guard
    words that must survive the run (catches out-of-range stores)."""
    dev = torch.device("cuda:0")
    xd = torch.from_numpy(X).to(dev)
    wd = torch.from_numpy(W).to(dev)
    bd = torch.from_numpy(B).to(dev) if B is not None else None
    d = binding.Conv2dDesc(tuple(X.shape), tuple(W.shape), pads=None if auto_pad != "NOTSET" else pads,
                           strides=strides, dilations=dilations, group=group, auto_pad=auto_pad,
                           has_bias=B is not None, fuse_relu=relu)
    numel = int(np.prod(d.y_shape))
    guard = 64
    buf = torch.full((numel + 2 * guard,), 12345.0, dtype=torch.float32, device=dev)
    yd = buf[guard:guard + numel].view(d.y_shape)
    d.run(xd, wd, bd, Y=yd)
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    if canary:
        assert bool((buf[:guard] == 12345.0).all()) and bool((buf[guard + numel:] == 12345.0).all()), \
            "store outside Y"
    fam = d.kernel_family
    d.close()
    return yd.cpu().numpy(), fam


def check_conv(binding, torch, X, W, B, *, relu=False, images=None, **kw):
    """Full-tensor comparison (or only the listed images) against the oracle."""
    got, fam = run_conv_gpu(binding, torch, X, W, B, relu=relu, **kw)
    if images is None:
        want, S = oracle.conv2d(X, W, B, relu=relu, **kw)
        ratio = worst_ratio(got, want, S)
    else:
        want, S = oracle.conv2d(np.ascontiguousarray(X[images]), W, B, relu=relu, **kw)
        ratio = worst_ratio(got[images], want, S)
    return ratio, fam


def run_gemm_gpu(binding, torch, A, B, C, **kw):
    dev = torch.device("cuda:0")
    ad, bd = torch.from_numpy(A).to(dev), torch.from_numpy(B).to(dev)
    cd = torch.from_numpy(np.ascontiguousarray(C)).to(dev) if C is not None else None
    y = binding.onnx_gemm(ad, bd, cd, **kw)
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    return y.cpu().numpy()
