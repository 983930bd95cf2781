"""Pins for the fp64 oracle: hand-computed cases, closed forms, algebraic identities,
a structurally different second route (explicit im2col), brute force in pure Python
and library cross-checks.  None of these re-type the oracle's loop nest."""
import itertools
import json
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")
with open(GOLDEN) as fh:
    HAND = json.load(fh)


# ---------------------------------------------------------------- hand-computed
@pytest.mark.parametrize("case", HAND["conv"], ids=lambda c: c["name"])
def test_conv_hand_cases(case):
    X = np.array(case["x"], np.float32).reshape(case["x_shape"])
    W = np.array(case["w"], np.float32).reshape(case["w_shape"])
    B = np.array(case["b"], np.float32) if "b" in case else None
    Y, S = oracle.conv2d(X, W, B, pads=case.get("pads", (0, 0, 0, 0)),
                         strides=case.get("strides", (1, 1)),
                         dilations=case.get("dilations", (1, 1)),
                         group=case.get("group", 1), relu=case.get("relu", False))
    assert list(Y.shape) == case["y_shape"]
    assert np.array_equal(Y.ravel(), np.array(case["y"], np.float64))
    assert (S >= 0).all()


@pytest.mark.parametrize("case", HAND["gemm"], ids=lambda c: c["name"])
def test_gemm_hand_cases(case):
    A = np.array(case["a"], np.float32).reshape(case["a_shape"])
    B = np.array(case["b"], np.float32).reshape(case["b_shape"])
    C = np.array(case["c"], np.float32).reshape(case["c_shape"]) if "c" in case else None
    Y, _ = oracle.gemm(A, B, C, alpha=case.get("alpha", 1.0), beta=case.get("beta", 1.0),
                       transA=case.get("transA", False), transB=case.get("transB", False),
                       relu=case.get("relu", False))
    assert list(Y.shape) == case["y_shape"]
    assert np.array_equal(Y.ravel(), np.array(case["y"], np.float64))


@pytest.mark.parametrize("case", HAND["same_pad"], ids=lambda c: c["name"])
def test_same_pad_hand_cases(case):
    # exercise the H axis and the W axis separately so that a swapped axis shows
    for axis in (0, 1):
        x = [1, 1, 3, 3]
        w = [1, 1, 1, 1]
        strides, dil = [1, 1], [1, 1]
        x[2 + axis], w[2 + axis] = case["in"], case["k"]
        strides[axis], dil[axis] = case["s"], case["d"]
        y, pads = oracle.conv2d_output_shape(x, w, strides=strides, dilations=dil,
                                             auto_pad=case["auto_pad"])
        assert y[2 + axis] == case["out"]
        assert pads[axis] == case["begin"] and pads[2 + axis] == case["end"]
        assert y[3 - axis] == 3 and pads[1 - axis] == 0 and pads[3 - axis] == 0


# ---------------------------------------------------------------- shape rules
def test_output_size_formula_and_errors():
    y, pads = oracle.conv2d_output_shape((2, 3, 224, 224), (64, 3, 7, 7), pads=(3, 3, 3, 3), strides=(2, 2))
    assert y == (2, 64, 112, 112) and pads == (3, 3, 3, 3)
    y, _ = oracle.conv2d_output_shape((1, 4, 10, 9), (6, 2, 3, 2), pads=(1, 0, 2, 1), strides=(3, 2),
                                      dilations=(2, 3), group=2)
    # H: 10+1+2-5 = 8 -> 8//3+1 = 3 ; W: 9+0+1-4 = 6 -> 6//2+1 = 4
    assert y == (1, 6, 3, 4)
    y, pads = oracle.conv2d_output_shape((1, 1, 5, 5), (1, 1, 3, 3), auto_pad="VALID")
    assert y == (1, 1, 3, 3) and pads == (0, 0, 0, 0)
    bad = [
        dict(x=(1, 3, 5, 5), w=(4, 2, 3, 3)),                       # C/g mismatch
        dict(x=(1, 4, 5, 5), w=(3, 2, 3, 3), group=2),              # M % g
        dict(x=(1, 4, 5, 5), w=(4, 4, 3, 3), kernel_shape=(2, 2)),  # kernel_shape vs W
        dict(x=(1, 4, 5, 5), w=(4, 4, 3, 3), strides=(0, 1)),
        dict(x=(1, 4, 5, 5), w=(4, 4, 3, 3), dilations=(1, -1)),
        dict(x=(1, 4, 5, 5), w=(4, 4, 3, 3), pads=(1, 1, 1, 1), auto_pad="SAME_UPPER"),
        dict(x=(1, 4, 2, 2), w=(4, 4, 3, 3)),                       # kernel larger than input
        dict(x=(1, 4, 5, 5), w=(4, 4, 3, 3), pads=(-1, 0, 0, 0)),
        dict(x=(1, 4, 5), w=(4, 4, 3, 3)),
    ]
    for kw in bad:
        kw = dict(kw)
        x, w = kw.pop("x"), kw.pop("w")
        with pytest.raises(oracle.OracleShapeError):
            oracle.conv2d_output_shape(x, w, **kw)


@given(size=st.integers(1, 40), k=st.integers(1, 5), s=st.integers(1, 4),
       mode=st.sampled_from(["SAME_UPPER", "SAME_LOWER"]))
@settings(max_examples=200, deadline=None)
def test_same_pad_invariants(size, k, s, mode):
    y, pads = oracle.conv2d_output_shape((1, 1, size, 3), (1, 1, k, 1), strides=(s, 1), auto_pad=mode)
    assert y[2] == -(-size // s)                          # out = ceil(in / stride)
    assert abs(pads[0] - pads[2]) <= 1
    assert (pads[0] <= pads[2]) if mode == "SAME_UPPER" else (pads[0] >= pads[2])
    # the resolved pads reproduce the same output size through the explicit formula
    y2, _ = oracle.conv2d_output_shape((1, 1, size, 3), (1, 1, k, 1), strides=(s, 1), pads=pads)
    assert y2 == y


# ---------------------------------------------------------------- closed forms
def _count_taps(H, k, pad_begin, stride, dil, p):
    return sum(1 for r in range(k) if 0 <= p * stride + r * dil - pad_begin < H)


def test_all_ones_counts_inbounds_taps():
    C, H, W, kH, kW = 3, 7, 6, 3, 2
    pads, strides, dil = (2, 1, 1, 0), (2, 1), (1, 2)
    X = np.ones((1, C, H, W), np.float32)
    Wt = np.ones((2, C, kH, kW), np.float32)
    Y, S = oracle.conv2d(X, Wt, pads=pads, strides=strides, dilations=dil)
    _, _, P, Q = Y.shape
    for p in range(P):
        for q in range(Q):
            want = C * _count_taps(H, kH, pads[0], strides[0], dil[0], p) * _count_taps(W, kW, pads[1], strides[1], dil[1], q)
            assert Y[0, 0, p, q] == want == Y[0, 1, p, q] == S[0, 0, p, q]
    Yv, _ = oracle.conv2d(X, Wt)                       # no padding: every output = C*kH*kW
    assert (Yv == C * kH * kW).all()


def test_delta_kernel_is_a_shifted_strided_copy():
    rng = np.random.default_rng(1)
    X = rng.integers(-2048, 2048, size=(2, 3, 9, 8)).astype(np.float32)
    kH, kW, pads, strides, dil = 3, 3, (1, 2, 0, 1), (2, 1), (1, 2)
    for (c, r, s) in [(0, 0, 0), (2, 1, 2), (1, 2, 1)]:
        Wt = np.zeros((1, 3, kH, kW), np.float32)
        Wt[0, c, r, s] = 1.0
        Y, _ = oracle.conv2d(X, Wt, pads=pads, strides=strides, dilations=dil)
        Xp = np.zeros((2, 3, 9 + pads[0] + pads[2], 8 + pads[1] + pads[3]), np.float64)
        Xp[:, :, pads[0]:pads[0] + 9, pads[1]:pads[1] + 8] = X
        P, Q = Y.shape[2:]
        want = Xp[:, c, r * dil[0]: r * dil[0] + (P - 1) * strides[0] + 1: strides[0],
                  s * dil[1]: s * dil[1] + (Q - 1) * strides[1] + 1: strides[1]]
        assert np.array_equal(Y[:, 0], want)


def test_linearity_in_x_and_w():
    rng = np.random.default_rng(2)
    X1, X2 = rng.standard_normal((2, 1, 4, 6, 5)).astype(np.float32)
    W1, W2 = rng.standard_normal((2, 4, 2, 3, 2)).astype(np.float32)
    kw = dict(pads=(1, 0, 1, 2), strides=(1, 2), group=2)
    Ya, _ = oracle.conv2d(X1, W1, **kw)
    Yb, _ = oracle.conv2d(X2, W1, **kw)
    # float32 sums are exactly representable in float64 and the oracle reads float32:
    # use power-of-two scaling (exact) rather than X1+X2 (which would round in float32)
    Y2, _ = oracle.conv2d((X1 * np.float32(4.0)), W1, **kw)
    assert np.allclose(Y2, 4.0 * Ya, rtol=1e-15, atol=0)
    Yw, _ = oracle.conv2d(X1, (W1 * np.float32(-0.5)), **kw)
    assert np.allclose(Yw, -0.5 * Ya, rtol=1e-15, atol=0)
    # additivity through channel concatenation: conv([X1|X2],[W1|W2]) = conv(X1,W1) + conv(X2,W2)
    k1 = dict(pads=(1, 0, 1, 2), strides=(1, 2))
    Xa, Xb = X1[:, :2], X2[:, 2:]
    Wa, Wb = W1[:, :2], W2[:, :2]
    Ycat, _ = oracle.conv2d(np.concatenate([Xa, Xb], 1), np.concatenate([Wa, Wb], 1), **k1)
    Ysum = oracle.conv2d(Xa, Wa, **k1)[0] + oracle.conv2d(Xb, Wb, **k1)[0]
    assert np.allclose(Ycat, Ysum, rtol=1e-13, atol=1e-13)
    assert Yb.shape == Ya.shape


def test_s_is_conv_of_absolute_values():
    rng = np.random.default_rng(3)
    X = rng.standard_normal((1, 4, 6, 6)).astype(np.float32)
    Wt = rng.standard_normal((4, 2, 3, 3)).astype(np.float32)
    _, S = oracle.conv2d(X, Wt, pads=(1, 1, 1, 1), group=2)
    Yabs, _ = oracle.conv2d(np.abs(X), np.abs(Wt), pads=(1, 1, 1, 1), group=2)
    assert np.allclose(S, Yabs, rtol=1e-14)
    A = rng.standard_normal((5, 7)).astype(np.float32)
    B = rng.standard_normal((7, 3)).astype(np.float32)
    _, Sg = oracle.gemm(A, B, alpha=-2.0)
    assert np.allclose(Sg, 2.0 * (np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64)), rtol=1e-14)


# ---------------------------------------------------------------- textbook reductions
def test_1x1_conv_is_gemm_per_image():
    rng = np.random.default_rng(4)
    N, C, H, W, M = 3, 5, 4, 6, 7
    X = rng.standard_normal((N, C, H, W)).astype(np.float32)
    Wt = rng.standard_normal((M, C, 1, 1)).astype(np.float32)
    Bv = rng.standard_normal((M,)).astype(np.float32)
    Y, S = oracle.conv2d(X, Wt, Bv)
    for n in range(N):
        Yg, Sg = oracle.gemm(Wt.reshape(M, C), X[n].reshape(C, H * W), Bv.reshape(M, 1))
        assert np.allclose(Y[n].reshape(M, H * W), Yg, rtol=1e-14, atol=1e-14)
        assert np.allclose(S[n].reshape(M, H * W), Sg, rtol=1e-14, atol=1e-14)


def test_group_is_concatenation_and_depthwise_is_per_channel():
    rng = np.random.default_rng(5)
    X = rng.standard_normal((2, 6, 5, 5)).astype(np.float32)
    Wt = rng.standard_normal((9, 2, 3, 3)).astype(np.float32)       # group 3: Cg=2, Mg=3
    Bv = rng.standard_normal((9,)).astype(np.float32)
    kw = dict(pads=(1, 1, 1, 1), strides=(2, 1))
    Y, _ = oracle.conv2d(X, Wt, Bv, group=3, **kw)
    parts = [oracle.conv2d(X[:, 2 * g:2 * g + 2], Wt[3 * g:3 * g + 3], Bv[3 * g:3 * g + 3], **kw)[0] for g in range(3)]
    assert np.array_equal(Y, np.concatenate(parts, axis=1))
    Wd = rng.standard_normal((6, 1, 3, 3)).astype(np.float32)
    Yd, _ = oracle.conv2d(X, Wd, group=6, **kw)
    for c in range(6):
        assert np.array_equal(Yd[:, c:c + 1], oracle.conv2d(X[:, c:c + 1], Wd[c:c + 1], **kw)[0])


def test_gemm_is_matmul_then_add():
    """Sec. 3.4.3: Gemm(m1, m2, m3) replaces Add(MatMul(m1, m2), m3)."""
    rng = np.random.default_rng(6)
    A = rng.standard_normal((6, 9)).astype(np.float32)
    B = rng.standard_normal((9, 4)).astype(np.float32)
    for cshape in [(), (1,), (4,), (1, 4), (6, 1), (1, 1), (6, 4)]:
        C = rng.standard_normal(cshape).astype(np.float32)
        Y, _ = oracle.gemm(A, B, C)
        want = A.astype(np.float64) @ B.astype(np.float64) + C.astype(np.float64)
        assert np.allclose(Y, want, rtol=1e-13, atol=1e-13)
    with pytest.raises(oracle.OracleShapeError):
        oracle.gemm(A, B, np.zeros((6,), np.float32))       # length M != N is not a row vector
    Ct = rng.standard_normal((4, 6)).astype(np.float32)
    Y, _ = oracle.gemm(B, A, Ct, transA=True, transB=True, alpha=0.25, beta=-3.0)
    want = 0.25 * (B.astype(np.float64).T @ A.astype(np.float64).T) - 3.0 * Ct.astype(np.float64)
    assert np.allclose(Y, want, rtol=1e-13, atol=1e-13)


# ---------------------------------------------------------------- second route: explicit im2col
def _im2col_route(X, Wt, Bv, pads, strides, dil, group):
    """Build the unfolded matrix with numpy indexing, contract with a float64 matmul."""
    N, C, H, W = X.shape
    M, Cg, kH, kW = Wt.shape
    (_, _, P, Q), pads = oracle.conv2d_output_shape(X.shape, Wt.shape, pads=pads, strides=strides,
                                                    dilations=dil, group=group)
    Xp = np.zeros((N, C, H + pads[0] + pads[2], W + pads[1] + pads[3]), np.float64)
    Xp[:, :, pads[0]:pads[0] + H, pads[1]:pads[1] + W] = X
    cols = np.empty((N, C, kH, kW, P, Q), np.float64)
    for r, s in itertools.product(range(kH), range(kW)):
        cols[:, :, r, s] = Xp[:, :, r * dil[0]: r * dil[0] + (P - 1) * strides[0] + 1: strides[0],
                              s * dil[1]: s * dil[1] + (Q - 1) * strides[1] + 1: strides[1]]
    Mg = M // group
    Y = np.empty((N, M, P, Q), np.float64)
    for g in range(group):
        a = Wt[g * Mg:(g + 1) * Mg].astype(np.float64).reshape(Mg, Cg * kH * kW)
        b = cols[:, g * Cg:(g + 1) * Cg].reshape(N, Cg * kH * kW, P * Q)
        Y[:, g * Mg:(g + 1) * Mg] = np.einsum("mk,nkp->nmp", a, b).reshape(N, Mg, P, Q)
    if Bv is not None:
        Y += Bv.astype(np.float64)[None, :, None, None]
    return Y


conv_problem = st.builds(
    dict,
    N=st.integers(1, 2), Cg=st.integers(1, 3), Mg=st.integers(1, 3), group=st.integers(1, 3),
    H=st.integers(1, 9), W=st.integers(1, 9), kH=st.integers(1, 4), kW=st.integers(1, 4),
    sh=st.integers(1, 3), sw=st.integers(1, 3), dh=st.integers(1, 3), dw=st.integers(1, 3),
    pt=st.integers(0, 3), pl=st.integers(0, 3), pb=st.integers(0, 3), pr=st.integers(0, 3),
    bias=st.booleans(), seed=st.integers(0, 2 ** 31 - 1),
)


@given(p=conv_problem)
@settings(max_examples=150, deadline=None)
def test_direct_definition_matches_im2col_route(p):
    eff_h, eff_w = (p["kH"] - 1) * p["dh"] + 1, (p["kW"] - 1) * p["dw"] + 1
    if p["H"] + p["pt"] + p["pb"] < eff_h or p["W"] + p["pl"] + p["pr"] < eff_w:
        return
    rng = np.random.default_rng(p["seed"])
    C, M = p["Cg"] * p["group"], p["Mg"] * p["group"]
    X = rng.standard_normal((p["N"], C, p["H"], p["W"])).astype(np.float32)
    Wt = rng.standard_normal((M, p["Cg"], p["kH"], p["kW"])).astype(np.float32)
    Bv = rng.standard_normal((M,)).astype(np.float32) if p["bias"] else None
    pads, strides, dil = (p["pt"], p["pl"], p["pb"], p["pr"]), (p["sh"], p["sw"]), (p["dh"], p["dw"])
    Y, _ = oracle.conv2d(X, Wt, Bv, pads=pads, strides=strides, dilations=dil, group=p["group"])
    want = _im2col_route(X, Wt, Bv, pads, strides, dil, p["group"])
    assert Y.shape == want.shape
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- brute force in pure Python
def test_pure_python_brute_force_tiny():
    rng = np.random.default_rng(7)
    N, C, H, W, M, kH, kW, g = 1, 4, 4, 5, 2, 2, 3, 2
    pads, (sh, sw), (dh, dw) = (1, 2, 0, 1), (2, 1), (2, 1)
    X = rng.integers(-3, 4, (N, C, H, W)).astype(np.float32)
    Wt = rng.integers(-3, 4, (M, C // g, kH, kW)).astype(np.float32)
    Y, _ = oracle.conv2d(X, Wt, pads=pads, strides=(sh, sw), dilations=(dh, dw), group=g)
    P, Q = Y.shape[2:]
    for m, p, q in itertools.product(range(M), range(P), range(Q)):
        tot = 0
        for c, r, s in itertools.product(range(C // g), range(kH), range(kW)):
            ih, iw = p * sh + r * dh - pads[0], q * sw + s * dw - pads[1]
            if 0 <= ih < H and 0 <= iw < W:
                tot += int(X[0, (m // (M // g)) * (C // g) + c, ih, iw]) * int(Wt[m, c, r, s])
        assert Y[0, m, p, q] == tot


# ---------------------------------------------------------------- library cross-checks
def test_against_torch_cpu_float64():
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    rng = np.random.default_rng(8)
    for (N, C, H, W, M, k, s, d, pad, g) in [(2, 4, 9, 8, 6, 3, 1, 1, 1, 1), (1, 6, 11, 10, 4, 3, 2, 2, 2, 2),
                                              (2, 3, 12, 12, 5, 7, 2, 1, 3, 1), (1, 8, 6, 6, 8, 3, 1, 1, 1, 8)]:
        X = rng.standard_normal((N, C, H, W)).astype(np.float32)
        Wt = rng.standard_normal((M, C // g, k, k)).astype(np.float32)
        Bv = rng.standard_normal((M,)).astype(np.float32)
        Y, _ = oracle.conv2d(X, Wt, Bv, pads=(pad,) * 4, strides=(s, s), dilations=(d, d), group=g)
        want = F.conv2d(torch.from_numpy(X).double(), torch.from_numpy(Wt).double(), torch.from_numpy(Bv).double(),
                        stride=s, padding=pad, dilation=d, groups=g).numpy()
        assert Y.shape == want.shape
        assert np.allclose(Y, want, rtol=1e-12, atol=1e-12)
    # asymmetric padding through an explicit F.pad (left, right, top, bottom)
    X = rng.standard_normal((1, 2, 5, 6)).astype(np.float32)
    Wt = rng.standard_normal((3, 2, 2, 3)).astype(np.float32)
    Y, _ = oracle.conv2d(X, Wt, pads=(2, 0, 1, 3))
    want = F.conv2d(F.pad(torch.from_numpy(X).double(), (0, 3, 2, 1)), torch.from_numpy(Wt).double()).numpy()
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-12)
    A = rng.standard_normal((7, 5)).astype(np.float32)
    B = rng.standard_normal((3, 5)).astype(np.float32)
    C = rng.standard_normal((3,)).astype(np.float32)
    Yg, _ = oracle.gemm(A, B, C, transB=True, alpha=1.5, beta=0.5)
    want = torch.addmm(torch.from_numpy(C).double(), torch.from_numpy(A).double(), torch.from_numpy(B).double().T,
                       beta=0.5, alpha=1.5).numpy()
    assert np.allclose(Yg, want, rtol=1e-13, atol=1e-13)


def test_relu_only_clamps_negatives():
    rng = np.random.default_rng(9)
    X = rng.standard_normal((1, 2, 5, 5)).astype(np.float32)
    Wt = rng.standard_normal((3, 2, 3, 3)).astype(np.float32)
    Y, _ = oracle.conv2d(X, Wt)
    Yr, _ = oracle.conv2d(X, Wt, relu=True)
    assert np.array_equal(Yr, np.maximum(Y, 0.0)) and (Y < 0).any()
