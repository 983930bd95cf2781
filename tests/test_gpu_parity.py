"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs.  Bar: |gpu - oracle| <= 1e-3 * sum|x*w| + 1e-5 per
output element; output shapes, index mapping and integer-valued cases bit-exact."""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2008_08272_b200 import workloads as wl

from parity import check_conv, run_conv_gpu, run_gemm_gpu, worst_ratio

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def binding():
    from paper_2008_08272_b200 import binding as b
    b.load(build_if_missing=False)      # the compiled library must be there: no fallback
    return b


with open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")) as fh:
    HAND = json.load(fh)


@pytest.mark.parametrize("case", HAND["conv"], ids=lambda c: c["name"])
def test_conv_hand_cases_bit_exact(binding, case):
    X = np.array(case["x"], np.float32).reshape(case["x_shape"])
    W = np.array(case["w"], np.float32).reshape(case["w_shape"])
    B = np.array(case["b"], np.float32) if "b" in case else None
    got, _ = run_conv_gpu(binding, torch, X, W, B, pads=case.get("pads", (0, 0, 0, 0)),
                          strides=case.get("strides", (1, 1)), dilations=case.get("dilations", (1, 1)),
                          group=case.get("group", 1), relu=case.get("relu", False))
    assert list(got.shape) == case["y_shape"]
    assert np.array_equal(got.ravel().astype(np.float64), np.array(case["y"], np.float64))


@pytest.mark.parametrize("case", HAND["gemm"], ids=lambda c: c["name"])
def test_gemm_hand_cases_bit_exact(binding, case):
    A = np.array(case["a"], np.float32).reshape(case["a_shape"])
    B = np.array(case["b"], np.float32).reshape(case["b_shape"])
    C = np.array(case["c"], np.float32).reshape(case["c_shape"]) if "c" in case else None
    got = run_gemm_gpu(binding, torch, A, B, C, alpha=case.get("alpha", 1.0), beta=case.get("beta", 1.0),
                       transA=case.get("transA", False), transB=case.get("transB", False),
                       fuse_relu=case.get("relu", False))
    assert np.array_equal(got.ravel().astype(np.float64), np.array(case["y"], np.float64))


def _random_conv_problems(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        g = int(rng.choice([1, 1, 1, 2, 3, 4]))
        Cg, Mg = int(rng.integers(1, 9)), int(rng.integers(1, 11))
        H, W = int(rng.integers(1, 24)), int(rng.integers(1, 24))
        kH, kW = int(rng.integers(1, 6)), int(rng.integers(1, 6))
        sh, sw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        dh, dw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        pads = tuple(int(v) for v in rng.integers(0, 4, 4))
        if H + pads[0] + pads[2] < (kH - 1) * dh + 1 or W + pads[1] + pads[3] < (kW - 1) * dw + 1:
            continue
        out.append(dict(N=int(rng.integers(1, 4)), C=Cg * g, M=Mg * g, Cg=Cg, H=H, W=W, kH=kH, kW=kW,
                        strides=(sh, sw), dilations=(dh, dw), pads=pads, group=g,
                        bias=bool(rng.integers(0, 2)), relu=bool(rng.integers(0, 2)), seed=int(rng.integers(1 << 30))))
    return out


@pytest.mark.parametrize("p", _random_conv_problems(60, 1234), ids=lambda p: "x".join(
    str(p[k]) for k in ("N", "C", "H", "W", "M", "kH", "kW", "group")))
def test_conv_random_small(binding, p):
    rng = np.random.default_rng(p["seed"])
    X = rng.standard_normal((p["N"], p["C"], p["H"], p["W"])).astype(np.float32)
    W = rng.standard_normal((p["M"], p["Cg"], p["kH"], p["kW"])).astype(np.float32)
    B = rng.standard_normal((p["M"],)).astype(np.float32) if p["bias"] else None
    ratio, _ = check_conv(binding, torch, X, W, B, relu=p["relu"], pads=p["pads"], strides=p["strides"],
                          dilations=p["dilations"], group=p["group"])
    assert ratio <= 1.0, ratio


# shapes that span several tiles of every kernel family and leave ragged tails
MID_CASES = [
    dict(x=(2, 32, 30, 30), w=(48, 32, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(3, 64, 17, 19), w=(96, 64, 1, 1)),
    dict(x=(2, 40, 29, 31), w=(72, 40, 1, 1), strides=(2, 2)),
    dict(x=(2, 24, 33, 35), w=(40, 24, 3, 3), pads=(1, 1, 1, 1), strides=(2, 2)),
    dict(x=(1, 16, 41, 37), w=(24, 16, 3, 3), pads=(2, 2, 2, 2), dilations=(2, 2)),
    dict(x=(2, 3, 67, 65), w=(32, 3, 7, 7), pads=(3, 3, 3, 3), strides=(2, 2)),
    dict(x=(2, 64, 20, 20), w=(64, 16, 3, 3), pads=(1, 1, 1, 1), group=4),
    dict(x=(2, 96, 27, 29), w=(96, 1, 3, 3), pads=(1, 1, 1, 1), group=96),
    dict(x=(2, 40, 31, 33), w=(40, 1, 5, 5), pads=(2, 2, 2, 2), strides=(2, 2), group=40),
    dict(x=(1, 128, 7, 7), w=(256, 128, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(2, 256, 14, 14), w=(128, 256, 1, 1)),
    dict(x=(2, 64, 56, 56), w=(256, 64, 1, 1)),
    dict(x=(3, 96, 20, 20), w=(40, 96, 1, 1)),
    dict(x=(2, 36, 12, 12), w=(130, 36, 1, 1)),
    dict(x=(1, 8, 9, 300), w=(16, 8, 1, 5), pads=(0, 2, 0, 2)),
    dict(x=(1, 8, 300, 9), w=(16, 8, 5, 1), pads=(2, 0, 2, 0)),
]


@pytest.mark.parametrize("c", MID_CASES, ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
@pytest.mark.parametrize("relu", [False, True])
def test_conv_multi_tile(binding, c, relu):
    rng = np.random.default_rng(77)
    X = rng.random(c["x"], dtype=np.float32)
    fan = c["w"][1] * c["w"][2] * c["w"][3]
    W = (rng.standard_normal(c["w"]) * np.sqrt(2.0 / fan)).astype(np.float32)
    B = (rng.standard_normal((c["w"][0],)) * 0.1).astype(np.float32)
    ratio, _ = check_conv(binding, torch, X, W, B, relu=relu, pads=c.get("pads", (0, 0, 0, 0)),
                          strides=c.get("strides", (1, 1)), dilations=c.get("dilations", (1, 1)),
                          group=c.get("group", 1))
    assert ratio <= 1.0, ratio


# the implicit-GEMM tensor-core kernel forced onto shapes the dispatcher would give to the SIMT
# family: thin contractions (tap-pair mode, C/group < 16), strides, dilations, groups, ragged sizes
FORCED_IMPLICIT = [
    dict(x=(2, 3, 64, 64), w=(32, 3, 7, 7), pads=(3, 3, 3, 3), strides=(2, 2)),
    dict(x=(2, 8, 32, 32), w=(24, 8, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(2, 4, 32, 32), w=(16, 4, 5, 5), pads=(2, 2, 2, 2)),
    dict(x=(2, 6, 36, 36), w=(20, 6, 3, 3), pads=(1, 1, 1, 1), strides=(2, 2)),
    dict(x=(2, 12, 32, 32), w=(20, 12, 3, 3), pads=(2, 2, 2, 2), dilations=(2, 2)),
    dict(x=(3, 2, 28, 28), w=(8, 2, 5, 5), pads=(2, 2, 2, 2)),
    dict(x=(2, 16, 24, 28), w=(40, 16, 3, 3), pads=(1, 0, 2, 1), strides=(2, 1)),
    dict(x=(2, 32, 20, 20), w=(48, 8, 3, 3), pads=(1, 1, 1, 1), group=4),
    dict(x=(5, 64, 7, 7), w=(70, 64, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(70, 4, 16, 16), w=(16, 4, 3, 3), pads=(1, 1, 1, 1)),
]


@pytest.mark.parametrize("c", FORCED_IMPLICIT, ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
def test_conv_forced_implicit_gemm(binding, c):
    rng = np.random.default_rng(4242)
    X = rng.standard_normal(c["x"]).astype(np.float32)
    W = rng.standard_normal(c["w"]).astype(np.float32)
    B = rng.standard_normal((c["w"][0],)).astype(np.float32)
    kw = dict(pads=c.get("pads", (0, 0, 0, 0)), strides=c.get("strides", (1, 1)),
              dilations=c.get("dilations", (1, 1)), group=c.get("group", 1))
    binding.set_kernel_override("mma_implicit")
    try:
        got, fam = run_conv_gpu(binding, torch, X, W, B, relu=True, **kw)
    finally:
        binding.set_kernel_override(None)
    assert fam == "mma_implicit"
    want, S = oracle.conv2d(X, W, B, relu=True, **kw)
    assert worst_ratio(got, want, S) <= 1.0


# every tile shape of the implicit-GEMM kernel, single CTA and CTA pair (cluster of two, M = 256
# instructions), on shapes with several tiles, a half-empty last pair tile, groups and ragged channels
TILE_CASES = [
    dict(x=(3, 32, 30, 30), w=(64, 32, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(5, 48, 14, 14), w=(272, 48, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(2, 64, 20, 20), w=(96, 16, 3, 3), pads=(1, 1, 1, 1), group=4),
    dict(x=(9, 32, 7, 7), w=(144, 32, 3, 3), pads=(1, 1, 1, 1)),
    dict(x=(2, 3, 64, 64), w=(64, 3, 7, 7), pads=(3, 3, 3, 3), strides=(2, 2)),
]


@pytest.mark.parametrize("tile", ["1,1,64", "1,2,64", "1,2,128", "1,1,256", "2,1,64", "2,2,64", "2,2,128", "2,1,256",
                                  "2,2,256", "2,1,48"])
@pytest.mark.parametrize("c", TILE_CASES, ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
def test_conv_implicit_gemm_tile_shapes(binding, c, tile, monkeypatch):
    rng = np.random.default_rng(99)
    X = rng.standard_normal(c["x"]).astype(np.float32)
    W = rng.standard_normal(c["w"]).astype(np.float32)
    B = rng.standard_normal((c["w"][0],)).astype(np.float32)
    kw = dict(pads=c.get("pads", (0, 0, 0, 0)), strides=c.get("strides", (1, 1)), group=c.get("group", 1))
    monkeypatch.setenv("ONNXB_CONV_TILE", tile)      # read when the descriptor is created
    binding.set_kernel_override("mma_implicit")
    try:
        got, fam = run_conv_gpu(binding, torch, X, W, B, relu=False, **kw)
    finally:
        binding.set_kernel_override(None)
    assert fam == "mma_implicit"
    want, S = oracle.conv2d(X, W, B, relu=False, **kw)
    assert worst_ratio(got, want, S) <= 1.0


@pytest.mark.parametrize("c", TILE_CASES + FORCED_IMPLICIT[:4], ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
def test_conv_implicit_gemm_four_epilogue_warps(binding, c, monkeypatch):
    """The implicit-GEMM kernel's form with four epilogue warps (the planner picks it for thin first
    layers only), forced onto ordinary shapes."""
    rng = np.random.default_rng(404)
    X = rng.standard_normal(c["x"]).astype(np.float32)
    W = rng.standard_normal(c["w"]).astype(np.float32)
    B = rng.standard_normal((c["w"][0],)).astype(np.float32)
    kw = dict(pads=c.get("pads", (0, 0, 0, 0)), strides=c.get("strides", (1, 1)),
              dilations=c.get("dilations", (1, 1)), group=c.get("group", 1))
    monkeypatch.setenv("ONNXB_CONV_EPI", "4")        # read when the descriptor is created
    binding.set_kernel_override("mma_implicit")
    try:
        got, fam = run_conv_gpu(binding, torch, X, W, B, relu=True, **kw)
    finally:
        binding.set_kernel_override(None)
    assert fam == "mma_implicit"
    want, S = oracle.conv2d(X, W, B, relu=True, **kw)
    assert worst_ratio(got, want, S) <= 1.0


@pytest.mark.parametrize("relay", ["0", "1"])
@pytest.mark.parametrize("stages", ["2,2", "3,2"])
@pytest.mark.parametrize("tile", ["2,1,64", "2,2,64"])
def test_conv_implicit_gemm_pair_stage_handover(binding, tile, stages, relay, monkeypatch):
    """CTA pairs: the odd CTA's "operand stage written" message straight from its transform warps or through
    its relay warp, with two and three operand stages, on a problem with several tiles per CTA pair (so
    that every barrier of the hand-over wraps its phase more than once)."""
    rng = np.random.default_rng(int(relay) * 7 + len(tile))
    xs, ws = (40, 32, 30, 30), (64, 32, 3, 3)            # 40 x 31 x 31 slots = 150 / 75 pair tiles of 256 / 512
    X = rng.standard_normal(xs).astype(np.float32)
    W = rng.standard_normal(ws).astype(np.float32)
    B = rng.standard_normal((ws[0],)).astype(np.float32)
    monkeypatch.setenv("ONNXB_CONV_TILE", tile)           # all three are read when the descriptor is created
    monkeypatch.setenv("ONNXB_CONV_STAGES", stages)
    monkeypatch.setenv("ONNXB_CONV_RELAY", relay)
    binding.set_kernel_override("mma_implicit")
    try:
        got, fam = run_conv_gpu(binding, torch, X, W, B, relu=True, pads=(1, 1, 1, 1))
    finally:
        binding.set_kernel_override(None)
    assert fam == "mma_implicit"
    want, S = oracle.conv2d(X, W, B, relu=True, pads=(1, 1, 1, 1))
    assert worst_ratio(got, want, S) <= 1.0


@pytest.mark.parametrize("pair", ["0", "1"])
@pytest.mark.parametrize("shape", [(256, 200, 96), (384, 3136, 64), (300, 260, 130), (512, 64, 1024)])
def test_gemm_cta_pair_choice(binding, shape, pair, monkeypatch):
    """The tensor-core GEMM with one CTA per tile and with CTA pairs (256-row tiles), forced."""
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((K, N)).astype(np.float32)
    C = rng.standard_normal((N,)).astype(np.float32)
    monkeypatch.setenv("ONNXB_GEMM_PAIR", pair)
    got = run_gemm_gpu(binding, torch, A, B, C)
    want, S = oracle.gemm(A, B, C)
    assert worst_ratio(got, want, S) <= 1.0


@pytest.mark.parametrize("pair", ["0", "1"])
def test_conv1x1_cta_pair_choice(binding, pair, monkeypatch):
    """1x1 convolutions (direct and strided) through the GEMM kernel with the pair choice forced."""
    rng = np.random.default_rng(31)
    monkeypatch.setenv("ONNXB_GEMM_PAIR", pair)
    for xs, ws, st in [((3, 64, 14, 14), (320, 64, 1, 1), (1, 1)), ((2, 96, 28, 28), (256, 96, 1, 1), (2, 2)),
                       ((5, 128, 7, 7), (384, 128, 1, 1), (1, 1))]:
        X = rng.random(xs, dtype=np.float32)
        W = (rng.standard_normal(ws) * np.sqrt(2.0 / ws[1])).astype(np.float32)
        B = (rng.standard_normal((ws[0],)) * 0.1).astype(np.float32)
        ratio, _ = check_conv(binding, torch, X, W, B, relu=True, strides=st)
        assert ratio <= 1.0, (xs, ws, st, ratio)


def test_conv_auto_pad_and_no_bias(binding):
    rng = np.random.default_rng(5)
    X = rng.standard_normal((2, 6, 13, 11)).astype(np.float32)
    W = rng.standard_normal((4, 6, 4, 3)).astype(np.float32)
    for mode in ("SAME_UPPER", "SAME_LOWER", "VALID"):
        got, _ = run_conv_gpu(binding, torch, X, W, None, strides=(2, 3), auto_pad=mode)
        want, S = oracle.conv2d(X, W, None, strides=(2, 3), auto_pad=mode)
        assert worst_ratio(got, want, S) <= 1.0


def test_delta_kernel_index_mapping_bit_exact(binding):
    """A one-hot kernel turns Conv into a strided, shifted copy of one input channel.
    With integer codes |v| <= 2048 (exact in TF32 and fp32) the result must be bit-exact."""
    rng = np.random.default_rng(11)
    N, C, H, W = 3, 20, 37, 41
    X = rng.integers(-2048, 2049, size=(N, C, H, W)).astype(np.float32)
    for (M, k, s, d, pad, g) in [(8, 3, 1, 1, 1, 1), (12, 3, 2, 1, 1, 1), (4, 5, 1, 2, 4, 1), (20, 3, 1, 1, 1, 20),
                                 (10, 1, 2, 1, 0, 1), (40, 3, 1, 1, 1, 5)]:
        Cg = C // g
        Wt = np.zeros((M, Cg, k, k), np.float32)
        for m in range(M):
            Wt[m, (3 * m + 1) % Cg, (m + 1) % k, (2 * m) % k] = 1.0
        got, _ = run_conv_gpu(binding, torch, X, Wt, None, pads=(pad,) * 4, strides=(s, s), dilations=(d, d), group=g)
        want, _ = oracle.conv2d(X, Wt, None, pads=(pad,) * 4, strides=(s, s), dilations=(d, d), group=g, want_s=False)
        assert np.array_equal(got.astype(np.float64), want)


GEMM_CASES = [
    # M, N, K, transA, transB, c_shape, alpha, beta, relu
    (1, 1, 1, False, False, None, 1.0, 1.0, False),
    (5, 7, 3, False, False, (), 1.0, 1.0, False),
    (64, 10, 256, False, True, (10,), 1.0, 1.0, False),
    (65, 130, 70, True, False, (1, 130), 0.5, -2.0, True),
    (129, 67, 257, True, True, (129, 1), -1.5, 0.25, False),
    (200, 136, 96, False, True, (200, 136), 1.0, 1.0, True),
    (256, 384, 512, False, False, (384,), 1.0, 0.0, False),
    (300, 300, 64, False, True, (300,), 2.0, 1.0, False),
    (128, 1000, 2048, False, True, (1000,), 1.0, 1.0, False),
    (96, 40, 1030, True, False, (1,), 1.0, 3.0, False),
    (256, 512, 128, True, False, (256, 512), 1.0, 1.0, True),
    (384, 96, 200, True, True, (96,), 0.5, 1.0, False),
    (100, 260, 36, False, False, None, 1.0, 1.0, False),
    (128, 256, 32, False, True, None, 1.0, 1.0, False),
    (1000, 2500, 520, False, True, (2500,), 1.0, 1.0, True),
    (70, 33, 48, False, False, (1, 1), 1.0, -0.5, False),
    (256, 128, 64, False, True, (1, 1), 2.0, 1.0, True),
]


@pytest.mark.parametrize("c", GEMM_CASES, ids=lambda c: f"{c[0]}x{c[1]}x{c[2]}_{int(c[3])}{int(c[4])}")
def test_gemm_cases(binding, c):
    M, N, K, tA, tB, cshape, alpha, beta, relu = c
    rng = np.random.default_rng(M * 1000003 + N * 1009 + K)
    A = rng.standard_normal((K, M) if tA else (M, K)).astype(np.float32)
    B = rng.standard_normal((N, K) if tB else (K, N)).astype(np.float32)
    C = rng.standard_normal(cshape).astype(np.float32) if cshape is not None else None
    got = run_gemm_gpu(binding, torch, A, B, C, alpha=alpha, beta=beta, transA=tA, transB=tB, fuse_relu=relu)
    want, S = oracle.gemm(A, B, C, alpha=alpha, beta=beta, transA=tA, transB=tB, relu=relu)
    assert worst_ratio(got, want, S) <= 1.0


@pytest.mark.parametrize("pair", ["0", "1"])
@pytest.mark.parametrize("transB", [False, True])
@pytest.mark.parametrize("N", [68, 196, 264, 520, 784, 1028])
def test_gemm_narrow_last_tile(binding, N, transB, pair, monkeypatch):
    """The last tile along N is only as wide as the columns left (rounded up to 16), and the two CTAs of a
    pair split THAT width: 4 columns left (the second CTA then has none), 196 = one narrow tile whose second
    half starts off a 32-column block, 8 and 16 columns past full tiles, with a ragged K."""
    monkeypatch.setenv("ONNXB_GEMM_PAIR", pair)
    M, K = 300, 70
    rng = np.random.default_rng(N * 7 + int(transB))
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((N, K) if transB else (K, N)).astype(np.float32)
    C = rng.standard_normal((N,)).astype(np.float32)
    got = run_gemm_gpu(binding, torch, A, B, C, transB=transB, fuse_relu=True)
    want, S = oracle.gemm(A, B, C, transB=transB, relu=True)
    assert worst_ratio(got, want, S) <= 1.0


# ----------------------------------------------------------------- operands of one sign
# Every other case draws weights of mixed sign, whose TF32 operand errors largely cancel.  With X >= 0
# and W >= 0 nothing cancels: an operand the tensor core reads as stored loses its low 13 mantissa bits
# by truncation (one-sided, 3.4e-4 of the term on average, 9.8e-4 at most), a rounded one errs by at
# most 4.9e-4 either way.  The bar stays |err| <= 1e-3 * S + 1e-5.
def _same_sign_gemm(binding, M, N, K, transB):
    rng = np.random.default_rng(K * 31 + N)
    A = rng.random((M, K), dtype=np.float32)
    B = rng.random((N, K) if transB else (K, N), dtype=np.float32)
    got = run_gemm_gpu(binding, torch, A, B, None, transB=transB)
    want, S = oracle.gemm(A, B, None, transB=transB)
    return worst_ratio(got, want, S)


@pytest.mark.parametrize("K", [32, 64, 2048])
@pytest.mark.parametrize("transB", [False, True])
def test_gemm_same_sign_operands(binding, K, transB):
    ratio = _same_sign_gemm(binding, 192, 264, K, transB)
    print(f"same-sign Gemm K={K} transB={transB}: worst err/tol {ratio:.3f}")
    assert ratio <= 1.0, ratio


@pytest.mark.parametrize("transB", [False, True])
def test_gemm_same_sign_operands_split_k(binding, transB):
    """The classifier-head shape takes the split-K kernel, which rounds its operands itself in shared memory."""
    ratio = _same_sign_gemm(binding, 64, 1000, 2048, transB)
    print(f"same-sign split-K Gemm 64x1000x2048 transB={transB}: worst err/tol {ratio:.3f}")
    assert ratio <= 1.0, ratio


@pytest.mark.parametrize("shape", ["32,2", "32,4", "64,4", "64,8"])
@pytest.mark.parametrize("transB", [False, True])
def test_gemm_split_k_shapes(binding, shape, transB, monkeypatch):
    """Every tile width and cluster size of the split-K kernel, forced onto a ragged problem (M, N and K
    no multiples of the tile; the last cluster rank gets a short share of K), with C, alpha, beta and Relu."""
    monkeypatch.setenv("ONNXB_GEMM_SPLITK", shape)
    M, N, K = 100, 300, 1000
    rng = np.random.default_rng(77 + len(shape))
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((N, K) if transB else (K, N)).astype(np.float32)
    C = rng.standard_normal((M, 1)).astype(np.float32)
    got = run_gemm_gpu(binding, torch, A, B, C, alpha=0.5, beta=-1.5, transB=transB, fuse_relu=True)
    want, S = oracle.gemm(A, B, C, alpha=0.5, beta=-1.5, transB=transB, relu=True)
    assert worst_ratio(got, want, S) <= 1.0


SAME_SIGN_CONVS = [
    dict(x=(2, 64, 28, 28), w=(256, 64, 1, 1)),                          # 1x1 stride 1: X straight from NCHW
    dict(x=(2, 256, 28, 28), w=(64, 256, 1, 1)),
    dict(x=(2, 256, 28, 28), w=(128, 256, 1, 1), strides=(2, 2)),         # strided 1x1
    dict(x=(4, 256, 7, 7), w=(512, 256, 1, 1)),                           # 7x7 planes
    dict(x=(2, 64, 28, 28), w=(64, 64, 3, 3), pads=(1, 1, 1, 1)),         # implicit GEMM: both operands rounded
    dict(x=(2, 3, 64, 64), w=(64, 3, 7, 7), pads=(3, 3, 3, 3), strides=(2, 2)),
]


@pytest.mark.parametrize("c", SAME_SIGN_CONVS, ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
def test_conv_same_sign_operands(binding, c):
    rng = np.random.default_rng(606)
    X = rng.random(c["x"], dtype=np.float32)
    W = rng.random(c["w"], dtype=np.float32)
    B = rng.random((c["w"][0],), dtype=np.float32)
    ratio, fam = check_conv(binding, torch, X, W, B, relu=True, pads=c.get("pads", (0, 0, 0, 0)),
                            strides=c.get("strides", (1, 1)))
    print(f"same-sign conv {c['x']}x{c['w']} [{fam}]: worst err/tol {ratio:.3f}")
    assert ratio <= 1.0, (ratio, fam)


def test_conv_operands_just_above_a_tf32_grid_point(binding):
    """Activations whose mantissas sit just above a 10-bit grid point (1 + 2^-10 - 2^-23 times a power of
    two): the worst case for an operand that is truncated, harmless for one that is rounded.  Weights are
    exact in TF32, so the error is the activations' alone; kernels that round them are exact here, and the
    one path that reads X as stored (1x1, stride 1, by TMA) stays inside its documented bound of 1e-3 * S
    for X's part (2^-10 * S = 9.8e-4 * S)."""
    rng = np.random.default_rng(707)
    base = np.float32(1.0 + 2.0 ** -10 - 2.0 ** -23)
    for c in SAME_SIGN_CONVS:
        X = (base * np.exp2(rng.integers(-3, 3, size=c["x"]))).astype(np.float32)
        W = rng.integers(1, 9, size=c["w"]).astype(np.float32) / np.float32(8.0)
        ratio, fam = check_conv(binding, torch, X, W, None, pads=c.get("pads", (0, 0, 0, 0)),
                                strides=c.get("strides", (1, 1)))
        print(f"grid-point conv {c['x']}x{c['w']} [{fam}]: worst err/tol {ratio:.3f}")
        assert ratio <= 1.0, (ratio, fam)


# ----------------------------------------------------------------- the five configurations
def test_config1_mnist_conv(binding):
    case = wl.config1_mnist_conv()
    X, W, B = wl.conv_inputs(case)
    ratio, fam = check_conv(binding, torch, X, W, B, relu=case.relu, **_kw(case))
    assert ratio <= 1.0, (ratio, fam)


def test_config2_gemm_head(binding):
    case = wl.config2_gemm_head()
    A, B, C = wl.gemm_inputs(case)
    got = run_gemm_gpu(binding, torch, A, B, C, alpha=case.alpha, beta=case.beta, transA=case.transA,
                       transB=case.transB, fuse_relu=case.relu)
    want, S = oracle.gemm(A, B, C, alpha=case.alpha, beta=case.beta, transA=case.transA, transB=case.transB,
                          relu=case.relu)
    assert got.shape == (64, 10)
    assert worst_ratio(got, want, S) <= 1.0


def _kw(case):
    return dict(pads=case.pads, strides=case.strides, dilations=case.dilations, group=case.group)


def test_config3_stage2_3x3_full_tensor(binding):
    case = wl.config3_stage2_3x3()
    X, W, B = wl.conv_inputs(case)
    ratio, fam = check_conv(binding, torch, X, W, B, relu=case.relu, **_kw(case))
    assert ratio <= 1.0, (ratio, fam)


@pytest.mark.parametrize("idx", [0, 1])
def test_config4_stem_and_projection_full_tensor(binding, idx):
    case = wl.config4_stem_and_projection()[idx]
    X, W, B = wl.conv_inputs(case)
    ratio, fam = check_conv(binding, torch, X, W, B, relu=case.relu, **_kw(case))
    assert ratio <= 1.0, (ratio, fam)


def _unique_sweep_cases():
    seen, out = set(), []
    for c in wl.resnet50_v1_convs():
        key = (c.x_shape, c.w_shape, c.strides)
        if key not in seen:
            seen.add(key)
            out.append(c)
    return out + [wl.config5_depthwise()]


@pytest.mark.parametrize("case", _unique_sweep_cases(), ids=lambda c: c.name)
def test_config5_sweep_batch64_sampled_images(binding, case):
    """Full batch-64 launch (the configuration the benchmark times); the oracle checks
    images 0, 21, 42, 63 exactly (an image's outputs depend on that image only)."""
    X, W, B = wl.conv_inputs(case)
    ratio, fam = check_conv(binding, torch, X, W, B, relu=case.relu, images=[0, 21, 42, 63], **_kw(case))
    print(f"sweep {case.name} [{fam}]: worst err/tol {ratio:.3f}")
    assert ratio <= 1.0, (ratio, fam)


# (C, H = W, M, kernel, stride, pad, group): one shape per kernel family of the sweep
FULL_BATCH_INDEX_CASES = [
    (64, 56, 64, 3, 1, 1, 1),        # implicit GEMM, one CTA per tile
    (256, 56, 128, 1, 2, 0, 1),      # strided 1x1, one GEMM per image
    (512, 7, 512, 3, 1, 1, 1),       # implicit GEMM, CTA pairs, whole-image slabs
    (512, 7, 2048, 1, 1, 0, 1),      # 1x1 on 7x7 planes (49 pixels: no 16-byte row pitch), merged columns
    (1024, 14, 512, 1, 2, 0, 1),     # strided 1x1 onto 7x7 planes
    (256, 14, 1024, 1, 1, 0, 1),     # 1x1 straight on NCHW, CTA pairs
    (3, 224, 64, 7, 2, 3, 1),        # the stem: tap-pair mode, four parity planes
    (256, 28, 256, 3, 1, 1, 256),    # depthwise
]


@pytest.mark.parametrize("shape", FULL_BATCH_INDEX_CASES, ids=lambda t: "x".join(map(str, t)))
def test_sweep_index_mapping_on_full_batch(binding, shape):
    """Delta kernels on full batch-64 tensors, one sweep shape per kernel family: bit-exact copy
    semantics pin the index mapping of every image, not only the sampled ones."""
    C, HW, M, k, s, p, g = shape
    rng = np.random.default_rng(99 + C + HW)
    X = rng.integers(-1024, 1025, size=(64, C, HW, HW)).astype(np.float32)
    Cg = C // g
    Wt = np.zeros((M, Cg, k, k), np.float32)
    sel = [((5 * m + 3) % Cg, (m + 1) % k, (m // 2) % k) for m in range(M)]
    for m, (c, r, t) in enumerate(sel):
        Wt[m, c, r, t] = 1.0
    got, _ = run_conv_gpu(binding, torch, X, Wt, None, pads=(p,) * 4, strides=(s, s), group=g)
    Xp = np.zeros((64, C, HW + 2 * p, HW + 2 * p), np.float32)
    Xp[:, :, p:p + HW, p:p + HW] = X
    P = got.shape[2]
    assert P == (HW + 2 * p - k) // s + 1
    for m in range(0, M, 7):
        c, r, t = sel[m]
        cin = (m // (M // g)) * Cg + c
        want = Xp[:, cin, r:r + (P - 1) * s + 1:s, t:t + (P - 1) * s + 1:s]
        assert np.array_equal(got[:, m], want), (shape, m)


@pytest.mark.parametrize("shape,c_shape", [((64, 1000, 2048), (1000,)), ((130, 70, 300), (130, 1)), ((33, 40, 20), None)])
def test_matmul_add_entry(binding, shape, c_shape):
    """MatMul + Add through the fused entry (Sec. 3.4.3) against the oracle's Gemm with unit factors,
    which the CPU pins tie to MatMul followed by Add."""
    M, N, K = shape
    rng = np.random.default_rng(M * 7 + N)
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((K, N)).astype(np.float32)
    C = rng.standard_normal(c_shape).astype(np.float32) if c_shape else None
    dev = torch.device("cuda:0")
    y = binding.onnx_matmul_add(torch.from_numpy(A).to(dev), torch.from_numpy(B).to(dev),
                                torch.from_numpy(C).to(dev) if C is not None else None, fuse_relu=True)
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    want, S = oracle.gemm(A, B, C, relu=True)
    assert worst_ratio(y.cpu().numpy(), want, S) <= 1.0


# Conv + Add + Relu in one pass, one case per kernel family (and both GEMM store paths)
ADD_CASES = [
    dict(x=(2, 64, 28, 28), w=(256, 64, 1, 1)),                                   # GEMM, TMA stores, CTA pairs
    dict(x=(3, 96, 14, 14), w=(72, 96, 1, 1)),                                    # GEMM, one CTA per tile
    dict(x=(11, 64, 56, 56), w=(128, 64, 1, 1)),                                  # GEMM, one CTA, 256-wide tiles: one addend block in flight
    dict(x=(5, 128, 7, 7), w=(320, 128, 1, 1)),                                   # gathered, merged columns
    dict(x=(2, 64, 28, 28), w=(128, 64, 1, 1), strides=(2, 2)),                   # gathered, per image
    dict(x=(2, 32, 30, 30), w=(48, 32, 3, 3), pads=(1, 1, 1, 1)),                 # implicit GEMM
    dict(x=(9, 32, 7, 7), w=(144, 32, 3, 3), pads=(1, 1, 1, 1)),                  # implicit GEMM, pair tiles
    dict(x=(2, 4, 13, 11), w=(6, 4, 3, 3), pads=(1, 1, 1, 1)),                    # SIMT direct
    dict(x=(2, 24, 28, 28), w=(24, 1, 3, 3), pads=(1, 1, 1, 1), group=24),        # depthwise, unit stride
    dict(x=(2, 24, 27, 29), w=(24, 1, 5, 5), pads=(2, 2, 2, 2), strides=(2, 2), group=24),   # depthwise, general
]


@pytest.mark.parametrize("c", ADD_CASES, ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
@pytest.mark.parametrize("relu", [False, True])
def test_conv_add_relu_fused(binding, c, relu):
    """Y = relu?(Conv(X, W) + B + R) against the oracle's convolution plus the addend, Relu applied last."""
    rng = np.random.default_rng(515)
    X = rng.standard_normal(c["x"]).astype(np.float32)
    fan = c["w"][1] * c["w"][2] * c["w"][3]
    W = (rng.standard_normal(c["w"]) * np.sqrt(2.0 / fan)).astype(np.float32)
    B = (rng.standard_normal((c["w"][0],)) * 0.1).astype(np.float32)
    kw = dict(pads=c.get("pads", (0, 0, 0, 0)), strides=c.get("strides", (1, 1)), group=c.get("group", 1))
    conv, S = oracle.conv2d(X, W, B, relu=False, **kw)
    R = rng.standard_normal(conv.shape).astype(np.float32)
    want = conv + R.astype(np.float64)
    if relu:
        want = np.maximum(want, 0.0)
    dev = torch.device("cuda:0")
    d = binding.Conv2dDesc(tuple(X.shape), tuple(W.shape), has_bias=True, fuse_relu=relu, **kw)
    numel = want.size
    buf = torch.full((numel + 128,), 4321.0, dtype=torch.float32, device=dev)
    Y = buf[64:64 + numel].view(want.shape)
    d.run_add(torch.from_numpy(X).to(dev), torch.from_numpy(W).to(dev), torch.from_numpy(B).to(dev),
              torch.from_numpy(R).to(dev), Y=Y)
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    assert bool((buf[:64] == 4321.0).all()) and bool((buf[64 + numel:] == 4321.0).all()), "store outside Y"
    d.close()
    assert worst_ratio(Y.cpu().numpy(), want, S) <= 1.0


def test_conv_add_many_tiles_per_cta(binding):
    """The fused addend over a launch in which every CTA walks several tiles (the addend's blocks are
    requested ahead, across tile boundaries): sampled images against the oracle, which treats each
    image on its own, and the images in between against a second run on those images alone."""
    rng = np.random.default_rng(9917)
    n = 40
    X = rng.standard_normal((n, 64, 56, 56)).astype(np.float32)
    W = (rng.standard_normal((256, 64, 1, 1)) * np.sqrt(2.0 / 64)).astype(np.float32)
    B = (rng.standard_normal((256,)) * 0.1).astype(np.float32)
    R = rng.standard_normal((n, 256, 56, 56)).astype(np.float32)
    dev = torch.device("cuda:0")
    d = binding.Conv2dDesc(X.shape, W.shape, has_bias=True, fuse_relu=True)
    Xd, Wd, Bd, Rd = (torch.from_numpy(a).to(dev) for a in (X, W, B, R))
    Y = d.run_add(Xd, Wd, Bd, Rd)
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    d.close()
    pick = [0, 17, n - 1]
    conv, S = oracle.conv2d(X[pick], W, B, relu=False)
    want = np.maximum(conv + R[pick].astype(np.float64), 0.0)
    assert worst_ratio(Y[pick].cpu().numpy(), want, S) <= 1.0
    # the same arithmetic on a three-image launch: identical bits image by image
    d3 = binding.Conv2dDesc(X[pick].shape, W.shape, has_bias=True, fuse_relu=True)
    Y3 = d3.run_add(Xd[pick].contiguous(), Wd, Bd, Rd[pick].contiguous())
    torch.cuda.synchronize()
    d3.close()
    assert torch.equal(Y3, Y[pick])


@pytest.mark.parametrize("c", [ADD_CASES[0], ADD_CASES[4], ADD_CASES[5], ADD_CASES[6], ADD_CASES[8]],
                         ids=lambda c: "x".join(map(str, c["x"] + c["w"])))
@pytest.mark.parametrize("with_r", [False, True])
def test_conv_prepacked_matches_the_plain_calls(binding, c, with_r):
    """Packing constant weights once and running from the copy gives bit for bit what the calls that
    pack at every run give (same kernels, same arithmetic)."""
    rng = np.random.default_rng(808)
    dev = torch.device("cuda:0")
    X = torch.from_numpy(rng.standard_normal(c["x"]).astype(np.float32)).to(dev)
    W = torch.from_numpy((rng.standard_normal(c["w"]) * 0.1).astype(np.float32)).to(dev)
    B = torch.from_numpy(rng.standard_normal((c["w"][0],)).astype(np.float32)).to(dev)
    kw = dict(pads=c.get("pads", (0, 0, 0, 0)), strides=c.get("strides", (1, 1)), group=c.get("group", 1))
    d = binding.Conv2dDesc(c["x"], c["w"], has_bias=True, fuse_relu=True, **kw)
    R = torch.from_numpy(rng.standard_normal(d.y_shape).astype(np.float32)).to(dev) if with_r else None
    want = d.run_add(X, W, B, R) if with_r else d.run(X, W, B)
    packed = d.prepack(W)
    got = d.run_prepacked(X, W, packed, B, R)
    got2 = d.run_prepacked(X, W, packed, B, R)          # the copy is read only: a second run finds it intact
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    assert torch.equal(got, want) and torch.equal(got2, want)
    d.close()


def test_tf32_mma_rate_probe(binding):
    """The measurement aid returns a plausible figure: never faster than the tensor pipe's ideal
    n/2 cycles per 128 x n x 8 instruction, and within a factor two of it; bad arguments are refused."""
    for n in (64, 256):
        cyc = binding.probe_tf32_mma_rate(n, 1024)
        assert n / 2 * 0.98 <= cyc <= n, (n, cyc)
    with pytest.raises(binding.OnnxB200Error):
        binding.probe_tf32_mma_rate(100, 1024)
    assert binding.last_device_status() == 0


def test_run_rejects_short_workspace_and_host_tensors(binding):
    x = torch.zeros((1, 4, 8, 8), device="cuda")
    w = torch.zeros((4, 4, 3, 3), device="cuda")
    with pytest.raises(TypeError):
        binding.onnx_conv2d(x.cpu(), w)
    y = binding.onnx_conv2d(x, w)
    assert y.shape == (1, 4, 6, 6) and float(y.abs().max()) == 0.0


def test_bounded_wait_runs_out_and_the_context_stays_usable(binding):
    """A device-side wait that nothing satisfies gives up after its limit, the kernel returns normally,
    the host sees ERR_DEVICE_TIMEOUT exactly once, and ordinary work afterwards is correct."""
    assert binding.last_device_status() == 0
    binding.probe_wait_timeout(1_000_000)                  # about half a millisecond of SM clock
    status = binding.last_device_status()
    assert binding.STATUS_NAMES[status] == "ERR_DEVICE_TIMEOUT"
    assert binding.last_device_status() == 0               # reading the word cleared it
    with pytest.raises(binding.OnnxB200Error):
        binding.probe_wait_timeout(0)
    rng = np.random.default_rng(3)
    X = rng.standard_normal((2, 32, 20, 20)).astype(np.float32)
    W = rng.standard_normal((48, 32, 3, 3)).astype(np.float32)
    ratio, fam = check_conv(binding, torch, X, W, None, pads=(1, 1, 1, 1))
    assert fam == "mma_implicit" and ratio <= 1.0
    assert binding.last_device_status() == 0
