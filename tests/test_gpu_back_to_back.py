"""Operators launched back to back on one stream, each reading what the one before wrote and writing over
what the one before read (two ping-pong buffers), with no host synchronisation in between.  The tensor-core
kernels start while the previous kernel is still draining (programmatic stream serialization) and only some
of their warps wait for it, so this is where an access in front of that wait would show: the result must be
bit-identical to the same chain run with a device synchronisation after every operator (same kernels, same
order of additions), and that run is compared with the oracle operator by operator."""
import numpy as np
import pytest

import oracle

from parity import worst_ratio

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _chain(binding, dev, rng, N, C, H):
    """(descriptor, weights, bias, packed weights, workspace, oracle arguments) per operator: an implicit-GEMM
    3x3, a 1x1 straight from NCHW, a depthwise 3x3 (a plainly launched SIMT kernel between two
    programmatically launched ones) and a 1x1 with a residual addend (the third buffer of the rotation)."""
    specs = [((C, C, 3, 3), dict(pads=(1, 1, 1, 1)), False), ((C, C, 1, 1), dict(), False),
             ((C, 1, 3, 3), dict(pads=(1, 1, 1, 1), group=C), False), ((C, C, 1, 1), dict(), True)]
    ops = []
    for ws, kw, with_r in specs:
        fan = ws[1] * ws[2] * ws[3]
        W = (rng.standard_normal(ws) * np.sqrt(1.0 / fan)).astype(np.float32)
        B = (rng.standard_normal((ws[0],)) * 0.05).astype(np.float32)
        d = binding.Conv2dDesc((N, C, H, H), ws, has_bias=True, fuse_relu=True, **kw)
        Wd, Bd = torch.from_numpy(W).to(dev), torch.from_numpy(B).to(dev)
        packed = d.prepack(Wd) if d.kernel_family in binding.WEIGHT_COPY_FAMILIES else None
        wsp = torch.empty(max(d.workspace_bytes, 16), dtype=torch.uint8, device=dev)
        ops.append((d, Wd, Bd, packed, wsp, W, B, kw, with_r))
    return ops


def _run(ops, x, rounds, sync):
    # three buffers in rotation: an operator reads the one written just before, writes over the one read
    # two operators ago, and takes its residual addend (when it has one) from the third
    bufs = [x.clone(), torch.zeros_like(x), torch.zeros_like(x)]
    outs = []
    cur = 0
    for _ in range(rounds):
        for d, Wd, Bd, packed, wsp, _, _, _, with_r in ops:
            src, dst, third = bufs[cur], bufs[(cur + 1) % 3], bufs[(cur + 2) % 3]
            R = third if with_r else None
            r_host = third.cpu().numpy() if (sync and with_r) else None
            if packed is not None:
                d.run_prepacked(src, Wd, packed, Bd, R, Y=dst, workspace=wsp)
            elif with_r:
                d.run_add(src, Wd, Bd, R, Y=dst, workspace=wsp)
            else:
                d.run(src, Wd, Bd, Y=dst, workspace=wsp)
            if sync:
                torch.cuda.synchronize()
                outs.append((src.cpu().numpy(), dst.cpu().numpy(), r_host))
            cur = (cur + 1) % 3
    torch.cuda.synchronize()
    return bufs[cur].clone(), outs


@pytest.mark.parametrize("shape", [(8, 64, 28), (1, 64, 14), (32, 128, 14)])
def test_back_to_back_chain_equals_the_synchronised_chain(shape):
    from paper_2008_08272_b200 import binding
    binding.load(build_if_missing=False)
    dev = torch.device("cuda:0")
    N, C, H = shape
    rng = np.random.default_rng(N * 100 + C + H)
    ops = _chain(binding, dev, rng, N, C, H)
    families = [o[0].kernel_family for o in ops]
    assert "mma_implicit" in families and "mma_gemm" in families and "simt_depthwise" in families
    x = torch.from_numpy(rng.random((N, C, H, H), dtype=np.float32)).to(dev)
    want, steps = _run(ops, x, rounds=1, sync=True)
    # the synchronised run against the oracle, operator by operator, on the inputs the chain gave it
    for (d, _, _, _, _, W, B, kw, with_r), (src, dst, r_host) in zip(ops, steps):
        ref, S = oracle.conv2d(src, W, B, relu=False, pads=kw.get("pads", (0, 0, 0, 0)), group=kw.get("group", 1))
        if with_r:
            ref = ref + r_host.astype(np.float64)
        ref = np.maximum(ref, 0.0)
        assert worst_ratio(dst, ref, S) <= 1.0, d.kernel_family
    want3, _ = _run(ops, x, rounds=3, sync=True)
    for _ in range(5):
        got3, _ = _run(ops, x, rounds=3, sync=False)
        assert binding.last_device_status() == 0
        assert torch.equal(got3, want3)
    for o in ops:
        o[0].close()
