"""onnx_conv2d_run_static is for callers that cannot allocate device memory (a frozen
memory budget, a host application that owns the allocator): it takes its scratch from an
array built into the library.  It must give what onnx_conv2d_run gives with a caller-made
workspace, bit for bit (the same kernels run), and that result must match the CPU oracle.
Collected last on purpose, so that a failure here cannot hide other results."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

REL, ABS = 1e-3, 1e-5      # the parity tolerance of the other GPU tests


# one layer per kernel family that uses scratch: packed weights (implicit GEMM), rounded weights
# (1x1 GEMM straight on NCHW), and whatever the strided 1x1 form keeps there
LAYERS = [
    ((2, 64, 28, 28), (96, 64, 3, 3), dict(pads=(1, 1, 1, 1))),
    ((3, 32, 14, 14), (40, 32, 3, 3), dict(pads=(1, 1, 1, 1), strides=(1, 1))),
    ((2, 64, 28, 28), (128, 64, 1, 1), dict(strides=(2, 2))),
    ((2, 64, 28, 28), (128, 64, 1, 1), dict()),
]


def test_static_scratch_entry_matches_workspace_entry_and_the_oracle():
    from paper_2008_08272_b200 import binding
    binding.load(build_if_missing=False)
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(2008)
    # different layers back to back, then the first again: every call finds the previous one's
    # leftovers in the shared array and must not be disturbed by them
    families = set()
    for call, (xs, ws, kw) in enumerate(LAYERS + LAYERS[:1]):
        Xh = rng.random(xs, dtype=np.float32)
        Wh = (rng.standard_normal(ws) * 0.05).astype(np.float32)
        Bh = (rng.standard_normal((ws[0],)) * 0.1).astype(np.float32)
        X, W, B = (torch.from_numpy(a).to(dev) for a in (Xh, Wh, Bh))
        d = binding.Conv2dDesc(xs, ws, has_bias=True, fuse_relu=True, **kw)
        assert d.workspace_bytes > 0, "the test must exercise kernels that really use scratch"
        assert d.workspace_bytes <= binding.static_scratch_bytes()
        families.add(d.kernel_family)
        want = d.run(X, W, B)                       # existing entry point, torch-allocated workspace
        got = torch.empty_like(want)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(dev)
        d.run_static(X, W, B, Y=got)                # new entry point, built-in scratch, output supplied
        d.run_static(X, W, B, Y=got)                # and again on top of its own leftovers
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before, "run_static must not allocate device memory"
        assert binding.last_device_status() == 0
        assert torch.equal(got, want), f"call {call} [{d.kernel_family}]: max diff {float((got - want).abs().max())}"
        ref, S = oracle.conv2d(Xh, Wh, Bh, relu=True, pads=kw.get("pads", (0, 0, 0, 0)),
                               strides=kw.get("strides", (1, 1)))
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
        assert (err <= REL * S + ABS).all(), f"call {call} [{d.kernel_family}]: worst ratio {(err / (REL * S + ABS)).max()}"
        d.close()
    assert "mma_implicit" in families and len(families) >= 2, families


def test_static_scratch_entry_rejects_oversized_layers():
    from paper_2008_08272_b200 import binding
    binding.load(build_if_missing=False)
    dev = torch.device("cuda:0")
    # 1024 x 1024 x 3 x 3 weights pack to 36 MiB, beyond the 10 MiB built-in array
    d = binding.Conv2dDesc((1, 1024, 8, 8), (1024, 1024, 3, 3), pads=(1, 1, 1, 1))
    assert d.workspace_bytes > binding.static_scratch_bytes()
    X = torch.zeros((1, 1024, 8, 8), device=dev)
    W = torch.zeros((1024, 1024, 3, 3), device=dev)
    before = binding.launch_count()
    with pytest.raises(binding.OnnxB200Error) as e:
        d.run_static(X, W)
    assert binding.STATUS_NAMES[e.value.status] == "ERR_WORKSPACE"
    assert binding.launch_count() == before         # nothing was launched
    d.close()
