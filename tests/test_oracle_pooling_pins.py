"""Pins of the pooling oracle (CPU): hand-computed cases, closed forms, pure-Python brute force and
torch's CPU routines, chosen so that a wrong pad side, a padded zero taking part in a maximum, a
ceil instead of a floor or a wrong divisor each fail at least one."""
import numpy as np
import pytest

import oracle


def test_maxpool_hand_case_pad_and_stride():
    # 1x1x3x4, kernel 2x2, stride 2, pads [0, 1, 0, 0] (one column on the LEFT only):
    # columns seen by q=0: {pad, 0}; q=1: {1, 2}; (q=2 would need column 3,4: W+pl-kW = 3 -> Q = 2)
    X = np.array([[[[-5, -1, -7, 4], [-2, -9, -3, -8], [6, 0, 1, 2]]]], np.float32)
    Y = oracle.maxpool2d(X, (2, 2), pads=(0, 1, 0, 0), strides=(2, 2))
    assert Y.shape == (1, 1, 1, 2)
    # p=0 covers rows 0,1.  q=0: max(-5, -2) = -2 (the pad is not a zero!), q=1: max(-1,-7,-9,-3) = -1
    assert Y.ravel().tolist() == [-2.0, -1.0]
    # a pad on the right instead would give Q = 2 with windows {0,1},{2,3}: max(-5,-1,-2,-9) = -1, max(-7,4,-3,-8) = 4
    Yr = oracle.maxpool2d(X, (2, 2), pads=(0, 0, 0, 1), strides=(2, 2))
    assert Yr.ravel().tolist() == [-1.0, 4.0]


def test_maxpool_output_size_is_floor():
    assert oracle.maxpool2d_output_shape((1, 1, 112, 112), (3, 3), (1, 1, 1, 1), (2, 2)) == (1, 1, 56, 56)
    assert oracle.maxpool2d_output_shape((1, 1, 7, 8), (2, 2), (0, 0, 0, 0), (2, 2)) == (1, 1, 3, 4)
    assert oracle.maxpool2d_output_shape((1, 1, 28, 28), (2, 2), (0, 0, 0, 0), (2, 2)) == (1, 1, 14, 14)
    with pytest.raises(oracle.PoolShapeError):
        oracle.maxpool2d_output_shape((1, 1, 2, 2), (3, 3))
    with pytest.raises(oracle.PoolShapeError):
        oracle.maxpool2d_output_shape((1, 1, 8, 8), (2, 2), (2, 0, 0, 0))


def test_maxpool_closed_forms():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((2, 3, 9, 11)).astype(np.float32)
    assert np.array_equal(oracle.maxpool2d(X, (1, 1)), X)                         # 1x1 window: identity
    assert np.array_equal(oracle.maxpool2d(np.full_like(X, -3.0), (3, 3), (1, 1, 1, 1), (2, 2)),
                          np.full((2, 3, 5, 6), -3.0, np.float32))                # all negative: pads must not win
    Yg = oracle.maxpool2d(X, (9, 11))                                             # whole image: the global maximum
    assert np.array_equal(Yg[:, :, 0, 0], X.max(axis=(2, 3)))
    Y = oracle.maxpool2d(X, (3, 3), (1, 1, 1, 1), (1, 1))
    assert Y.shape == X.shape and (Y >= X).all()                                  # every pixel lies in its own window


def test_maxpool_brute_force_and_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(2)
    for (H, W, k, s, pads) in [(7, 9, (3, 3), (2, 2), (1, 1, 1, 1)), (8, 8, (2, 2), (2, 2), (0, 0, 0, 0)),
                               (10, 6, (3, 2), (1, 3), (2, 0, 1, 1)), (5, 5, (5, 5), (1, 1), (0, 0, 0, 0))]:
        X = rng.standard_normal((2, 2, H, W)).astype(np.float32)
        Y = oracle.maxpool2d(X, k, pads, s)
        N, C, P, Q = Y.shape
        for n in range(N):
            for c in range(C):
                for p in range(P):
                    for q in range(Q):
                        best = -np.inf
                        for r in range(k[0]):
                            for t in range(k[1]):
                                h, w = p * s[0] + r - pads[0], q * s[1] + t - pads[1]
                                if 0 <= h < H and 0 <= w < W:
                                    best = max(best, float(X[n, c, h, w]))
                        assert Y[n, c, p, q] == np.float32(best)
        if pads[0] == pads[2] and pads[1] == pads[3]:
            ref = torch.nn.functional.max_pool2d(torch.from_numpy(X), k, s, (pads[0], pads[1])).numpy()
            assert np.array_equal(Y, ref)


def test_global_average_pool_pins():
    torch = pytest.importorskip("torch")
    X = np.arange(2 * 3 * 2 * 5, dtype=np.float32).reshape(2, 3, 2, 5)
    Y, S = oracle.global_average_pool(X)
    assert Y.shape == (2, 3, 1, 1)
    assert Y[0, 0, 0, 0] == 4.5 and Y[1, 2, 0, 0] == 54.5                          # mean of 0..9, of 50..59
    assert np.allclose(oracle.global_average_pool(np.ones((1, 4, 7, 7), np.float32))[0], 1.0, atol=0)
    rng = np.random.default_rng(3)
    A = rng.standard_normal((2, 5, 7, 7)).astype(np.float32)
    B = rng.standard_normal((2, 5, 7, 7)).astype(np.float32)
    ya, yb = oracle.global_average_pool(A)[0], oracle.global_average_pool(B)[0]
    yab = oracle.global_average_pool((A.astype(np.float64) + 2 * B.astype(np.float64)).astype(np.float32))[0]
    assert np.allclose(yab, ya + 2 * yb, atol=1e-6)                               # linear (up to the fp32 input rounding)
    ref = torch.nn.functional.adaptive_avg_pool2d(torch.from_numpy(A).double(), 1).numpy()
    assert np.allclose(ya, ref, rtol=1e-14, atol=1e-15)
    # S (the scale of the parity tolerance) is the mean of magnitudes: hand values on a mixed-sign plane,
    # where a signed mean (0.5) and a sum of magnitudes (10) would both show
    Ym, Sm = oracle.global_average_pool(np.array([[[[-1.0, 2.0], [-3.0, 4.0]]]], np.float32))
    assert Ym[0, 0, 0, 0] == 0.5 and Sm[0, 0, 0, 0] == 2.5
    assert S[0, 0, 0, 0] == 4.5 and S[1, 2, 0, 0] == 54.5                          # non-negative planes: S = Y
