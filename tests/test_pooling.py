"""MaxPool and GlobalAveragePool: host shape logic against the oracle's (CPU), and GPU parity
through the C ABI.  MaxPool must be bit-exact (a maximum involves no rounding); GlobalAveragePool
within |err| <= 1e-5 * mean|x| + 1e-7 (fp32 accumulation of at most 12544 terms, 32 partial sums
and a shuffle tree: the worst-case relative error of the sum is below (HW/32 + 5) * 2^-24 < 3e-5
of sum|x|, in practice far smaller)."""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def binding():
    from paper_2008_08272_b200 import binding as b
    b.load(build_if_missing=False)
    return b


def test_maxpool_shape_matches_oracle_and_rejects_bad_attributes(binding):
    rng = np.random.default_rng(5)
    for _ in range(200):
        H, W = int(rng.integers(1, 40)), int(rng.integers(1, 40))
        k = (int(rng.integers(1, 6)), int(rng.integers(1, 6)))
        s = (int(rng.integers(1, 4)), int(rng.integers(1, 4)))
        pads = tuple(int(v) for v in rng.integers(0, 4, 4))
        try:
            want = oracle.maxpool2d_output_shape((2, 3, H, W), k, pads, s)
        except oracle.PoolShapeError:
            with pytest.raises(binding.OnnxB200Error):
                binding.maxpool2d_shape((2, 3, H, W), k, pads, s)
            continue
        assert binding.maxpool2d_shape((2, 3, H, W), k, pads, s) == want
    assert binding.maxpool2d_shape((1, 64, 112, 112), (3, 3), (1, 1, 1, 1), (2, 2)) == (1, 64, 56, 56)
    assert binding.maxpool2d_shape((1, 8, 28, 28), (2, 2), None, (2, 2)) == (1, 8, 14, 14)


POOL_CASES = [
    dict(x=(2, 3, 9, 11), k=(3, 3), pads=(1, 1, 1, 1), s=(2, 2)),
    dict(x=(1, 8, 28, 28), k=(2, 2), pads=None, s=(2, 2)),                       # the MNIST model's pool
    dict(x=(3, 5, 17, 33), k=(3, 2), pads=(2, 0, 1, 1), s=(1, 3)),
    dict(x=(2, 4, 7, 7), k=(7, 7), pads=None, s=(1, 1)),
    dict(x=(2, 16, 37, 41), k=(5, 5), pads=(2, 2, 2, 2), s=(1, 1)),
    dict(x=(4, 64, 112, 112), k=(3, 3), pads=(1, 1, 1, 1), s=(2, 2)),            # ResNet50's pool, 4 images
]


@pytest.mark.gpu
@pytest.mark.parametrize("c", POOL_CASES, ids=lambda c: "x".join(map(str, c["x"] + c["k"])))
def test_maxpool_bit_exact(binding, c):
    rng = np.random.default_rng(7)
    X = rng.standard_normal(c["x"]).astype(np.float32) - 1.0          # mostly negative: a padded zero would win
    want = oracle.maxpool2d(X, c["k"], c["pads"] or (0, 0, 0, 0), c["s"])
    dev = torch.device("cuda:0")
    numel = want.size
    buf = torch.full((numel + 128,), 777.0, dtype=torch.float32, device=dev)
    Y = buf[64:64 + numel].view(want.shape)
    binding.onnx_maxpool2d(torch.from_numpy(X).to(dev), c["k"], pads=c["pads"], strides=c["s"], Y=Y)
    torch.cuda.synchronize()
    assert bool((buf[:64] == 777.0).all()) and bool((buf[64 + numel:] == 777.0).all()), "store outside Y"
    assert np.array_equal(Y.cpu().numpy(), want)


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(2, 5, 7, 7), (64, 2048, 7, 7), (3, 7, 1, 1), (2, 3, 56, 56), (1, 2, 13, 100)])
def test_global_average_pool_parity(binding, shape):
    rng = np.random.default_rng(9)
    X = rng.standard_normal(shape).astype(np.float32) + 0.25
    want, S = oracle.global_average_pool(X)
    y = binding.onnx_global_average_pool(torch.from_numpy(X).to(torch.device("cuda:0")))
    torch.cuda.synchronize()
    got = y.cpu().numpy().astype(np.float64)
    assert got.shape == want.shape
    assert np.all(np.abs(got - want) <= 1e-5 * S + 1e-7)
