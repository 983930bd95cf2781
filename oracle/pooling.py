"""CPU oracle for the two pooling operators of the paper's models (Sec. 4.1 lists pooling among the
lowered operators; MNIST has a MaxPool, ResNet50 a 3x3/stride-2 MaxPool and a global AveragePool,
Sec. 4.2).  Test infrastructure only.  The paper gives no formula; the ONNX definitions are the reading:

  MaxPool (2-D, NCHW, dilation 1, ceil_mode 0):
      Y[n,c,p,q] = max over r < kH, s < kW of X[n,c, p*sh + r - pt, q*sw + s - pl],
      positions outside the image do not take part (padding counts as minus infinity),
      P = floor((H + pt + pb - kH) / sh) + 1, same for Q; pads = [h_begin, w_begin, h_end, w_end].
  GlobalAveragePool: Y[n,c,0,0] = (1 / (H*W)) * sum over h, w of X[n,c,h,w], evaluated in fp64.

Each function is that definition written out tap by tap with numpy slices; no blocking or reordering.
"""
from __future__ import annotations

import numpy as np


class PoolShapeError(ValueError):
    pass


def maxpool2d_output_shape(x_shape, kernel_shape, pads=(0, 0, 0, 0), strides=(1, 1)):
    N, C, H, W = (int(v) for v in x_shape)
    kH, kW = (int(v) for v in kernel_shape)
    pt, pl, pb, pr = (int(v) for v in pads)
    sh, sw = (int(v) for v in strides)
    if min(N, C, H, W) < 1 or kH < 1 or kW < 1 or sh < 1 or sw < 1 or min(pt, pl, pb, pr) < 0:
        raise PoolShapeError("bad MaxPool attributes")
    if max(pt, pb) >= kH or max(pl, pr) >= kW:
        raise PoolShapeError("a pad as large as the kernel would leave windows with no input at all")
    if H + pt + pb < kH or W + pl + pr < kW:
        raise PoolShapeError("kernel larger than the padded input")
    return (N, C, (H + pt + pb - kH) // sh + 1, (W + pl + pr - kW) // sw + 1)


def maxpool2d(X, kernel_shape, pads=(0, 0, 0, 0), strides=(1, 1)):
    """ONNX MaxPool by its definition.  Returns Y as float32 (a maximum involves no rounding)."""
    X = np.asarray(X, dtype=np.float32)
    N, C, P, Q = maxpool2d_output_shape(X.shape, kernel_shape, pads, strides)
    kH, kW = kernel_shape
    pt, pl, pb, pr = pads
    sh, sw = strides
    H, W = X.shape[2:]
    Xp = np.full((N, C, H + pt + pb, W + pl + pr), -np.inf, dtype=np.float32)
    Xp[:, :, pt:pt + H, pl:pl + W] = X
    Y = np.full((N, C, P, Q), -np.inf, dtype=np.float32)
    for r in range(kH):
        for s in range(kW):
            Y = np.maximum(Y, Xp[:, :, r:r + (P - 1) * sh + 1:sh, s:s + (Q - 1) * sw + 1:sw])
    return Y


def global_average_pool(X):
    """ONNX GlobalAveragePool in fp64.  Returns (Y [N,C,1,1] float64, S = mean of |x| per plane)."""
    X64 = np.asarray(X, dtype=np.float32).astype(np.float64)
    if X64.ndim != 4 or min(X64.shape) < 1:
        raise PoolShapeError("GlobalAveragePool wants a non-empty NCHW tensor")
    hw = X64.shape[2] * X64.shape[3]
    Y = X64.sum(axis=(2, 3), keepdims=True) / hw
    S = np.abs(X64).sum(axis=(2, 3), keepdims=True) / hw
    return Y, S
