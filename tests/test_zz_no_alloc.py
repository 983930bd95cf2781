"""onnx_conv2d_run_static is for callers that cannot allocate device memory (a frozen
memory budget, a host application that owns the allocator): it takes its scratch from an
array built into the library.  It must give what onnx_conv2d_run gives with a caller-made
workspace.  Collected last on purpose, so that a failure here cannot hide other results."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

REL, ABS = 1e-3, 1e-5      # the parity tolerance of the other GPU tests


def test_static_scratch_entry_matches_workspace_entry_twice():
    from paper_2008_08272_b200 import binding
    binding.load(build_if_missing=False)
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(2008)
    # two different layers back to back: the second call finds the first one's leftovers
    # in the shared array and must not be disturbed by them
    layers = [((2, 64, 28, 28), (96, 64, 3, 3), dict(pads=(1, 1, 1, 1))),
              ((3, 32, 14, 14), (40, 32, 3, 3), dict(pads=(1, 1, 1, 1), strides=(1, 1)))]
    for call, (xs, ws, kw) in enumerate(layers + layers[:1]):
        X = torch.from_numpy(rng.random(xs, dtype=np.float32)).to(dev)
        W = torch.from_numpy((rng.standard_normal(ws) * 0.05).astype(np.float32)).to(dev)
        B = torch.from_numpy((rng.standard_normal((ws[0],)) * 0.1).astype(np.float32)).to(dev)
        d = binding.Conv2dDesc(xs, ws, has_bias=True, fuse_relu=True, **kw)
        assert d.kernel_family == "mma_implicit" and d.workspace_bytes > 0, \
            "the test must exercise a kernel that really uses scratch"
        assert d.workspace_bytes <= binding.static_scratch_bytes()
        want = d.run(X, W, B)                       # existing entry point, torch-allocated workspace
        got = d.run_static(X, W, B)                 # new entry point, built-in scratch
        torch.cuda.synchronize()
        assert binding.last_device_status() == 0
        # tolerance scale: sum |x*w| per output, from a plain fp32 convolution of magnitudes
        S = torch.nn.functional.conv2d(X.abs(), W.abs(), padding=1)
        err = (got - want).abs()
        assert bool((err <= REL * S + ABS).all()), f"call {call}: max err {float(err.max())}"
        d.close()


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
