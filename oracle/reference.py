"""Python face of the fp64 CPU oracle (test infrastructure only).

The arithmetic lives in ``onnx_oracle.c`` (plain C, one loop per index of the
defining sum, double precision).  This file holds the oracle's own shape and
padding rules for ONNX Conv, written separately from the product's descriptor
layer, and the ctypes marshalling.

The paper names convolution and Gemm as lowered operators (Sec. 4.1), infers
tensor shapes in a dedicated pass (Sec. 3.4.2) and defers operator semantics to
the ONNX standard (Sec. 2.1); the rules below are the reading of that standard
this repository follows.

Parity unpinned: NaN/Inf/-0 handling, and SAME_* padding with dilation > 1.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "onnx_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "libonnx_oracle.so")
_lock = threading.Lock()
_lib = None


class OracleShapeError(ValueError):
    """Attributes or shapes that ONNX Conv / Gemm do not admit."""


def build(force: bool = False) -> str:
    """Compile onnx_oracle.c with gcc (OpenMP) if the library is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB_PATH)
                 or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC))
        if force or stale:
            os.makedirs(_OUT_DIR, exist_ok=True)
            tmp = _LIB_PATH + ".%d.tmp" % os.getpid()
            subprocess.run(
                ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                 "-fno-fast-math", "-o", tmp, _SRC, "-lm"],
                check=True)
            os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, dbl, ptr = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.onnx_oracle_conv2d.restype = ctypes.c_int
        lib.onnx_oracle_conv2d.argtypes = [ptr, ptr, ptr] + [i64] * 16 + [ctypes.c_int, ptr, ptr]
        lib.onnx_oracle_gemm.restype = ctypes.c_int
        lib.onnx_oracle_gemm.argtypes = ([ptr, ptr, ptr] + [i64] * 3 + [ctypes.c_int] * 2
                                         + [dbl, dbl, i64, i64, ctypes.c_int, ptr, ptr])
        lib.onnx_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of host threads the C routines use (OpenMP default)."""
    return int(_load().onnx_oracle_threads())


def _pair(v, default, name):
    if v is None:
        return (default, default)
    v = tuple(int(t) for t in v)
    if len(v) != 2:
        raise OracleShapeError(f"{name} must have 2 entries")
    return v


def conv2d_output_shape(x_shape, w_shape, *, kernel_shape=None, pads=None, strides=None,
                        dilations=None, group=1, auto_pad="NOTSET"):
    """Shape inference for ONNX Conv (the Sec. 3.4.2 pass, restricted to one op).

    Returns ``(y_shape, pads)`` with ``pads = (h_begin, w_begin, h_end, w_end)``.

    Rules: out = floor((in + begin + end - ((k-1)*d + 1)) / stride) + 1;
    SAME_UPPER / SAME_LOWER choose out = ceil(in / stride) and the total padding
    max((out-1)*stride + (k-1)*d + 1 - in, 0), the odd unit going to the end for
    UPPER and to the beginning for LOWER; VALID means no padding; an auto_pad
    other than NOTSET may not be combined with explicit non-zero pads.
    """
    if len(x_shape) != 4 or len(w_shape) != 4:
        raise OracleShapeError("X and W must be rank 4")
    N, C, H, W = (int(t) for t in x_shape)
    M, Cg, kH, kW = (int(t) for t in w_shape)
    if min(N, C, H, W, M, Cg, kH, kW) < 1:
        raise OracleShapeError("empty dimension")
    if kernel_shape is not None and tuple(int(t) for t in kernel_shape) != (kH, kW):
        raise OracleShapeError("kernel_shape disagrees with W")
    sh, sw = _pair(strides, 1, "strides")
    dh, dw = _pair(dilations, 1, "dilations")
    if min(sh, sw, dh, dw) < 1:
        raise OracleShapeError("strides and dilations must be positive")
    group = int(group)
    if group < 1 or C % group or M % group or Cg * group != C:
        raise OracleShapeError("group does not divide the channel counts")
    if pads is None:
        pads = (0, 0, 0, 0)
    pads = tuple(int(t) for t in pads)
    if len(pads) != 4 or min(pads) < 0:
        raise OracleShapeError("pads must be 4 non-negative integers")
    eff = ((kH - 1) * dh + 1, (kW - 1) * dw + 1)
    if auto_pad != "NOTSET":
        if any(pads):
            raise OracleShapeError("auto_pad and explicit pads are exclusive")
        if auto_pad == "VALID":
            pads = (0, 0, 0, 0)
        elif auto_pad in ("SAME_UPPER", "SAME_LOWER"):
            begin, end = [], []
            for size, stride, e in ((H, sh, eff[0]), (W, sw, eff[1])):
                out = -(-size // stride)
                total = max((out - 1) * stride + e - size, 0)
                small, large = total // 2, total - total // 2
                if auto_pad == "SAME_UPPER":
                    begin.append(small), end.append(large)
                else:
                    begin.append(large), end.append(small)
            pads = (begin[0], begin[1], end[0], end[1])
        else:
            raise OracleShapeError(f"unknown auto_pad {auto_pad!r}")
    num_h = H + pads[0] + pads[2] - eff[0]
    num_w = W + pads[1] + pads[3] - eff[1]
    if num_h < 0 or num_w < 0:
        raise OracleShapeError("kernel larger than padded input")
    P, Q = num_h // sh + 1, num_w // sw + 1
    return (N, M, P, Q), pads


def conv2d(X, W, B=None, *, pads=(0, 0, 0, 0), strides=(1, 1), dilations=(1, 1), group=1,
           auto_pad="NOTSET", relu=False, want_s=True):
    """ONNX Conv by its definition, in fp64.  Returns ``(Y, S)`` (S is None if not wanted)."""
    X = np.ascontiguousarray(X, dtype=np.float32)
    W = np.ascontiguousarray(W, dtype=np.float32)
    y_shape, pads = conv2d_output_shape(X.shape, W.shape, pads=pads, strides=strides,
                                        dilations=dilations, group=group, auto_pad=auto_pad)
    sh, sw = _pair(strides, 1, "strides")
    dh, dw = _pair(dilations, 1, "dilations")
    if B is not None:
        B = np.ascontiguousarray(B, dtype=np.float32)
        if B.shape != (W.shape[0],):
            raise OracleShapeError("bias must have shape [M]")
    Y = np.empty(y_shape, dtype=np.float64)
    S = np.empty(y_shape, dtype=np.float64) if want_s else None
    N, C, H, Wd = X.shape
    M, _, kH, kW = W.shape
    rc = _load().onnx_oracle_conv2d(
        X.ctypes.data, W.ctypes.data, B.ctypes.data if B is not None else None,
        N, C, H, Wd, M, kH, kW, pads[0], pads[1], sh, sw, dh, dw, int(group),
        y_shape[2], y_shape[3], int(bool(relu)), Y.ctypes.data,
        S.ctypes.data if S is not None else None)
    if rc != 0:
        raise OracleShapeError("oracle rejected the group attribute")
    return Y, S


def gemm_c_strides(c_shape, M, N):
    """Element strides (along i, along j) of C broadcast one-directionally to [M,N].

    Admitted shapes: (), (1,), (N,), (1,N), (M,1), (M,N) and (1,1).  A 1-D C
    aligns with the trailing axis, so it is per-column even when M == N.
    """
    c_shape = tuple(int(t) for t in c_shape)
    if len(c_shape) > 2:
        raise OracleShapeError("C must have rank <= 2")
    full = (1,) * (2 - len(c_shape)) + c_shape
    if full[0] not in (1, M) or full[1] not in (1, N):
        raise OracleShapeError(f"C of shape {c_shape} does not broadcast to ({M},{N})")
    stride_i = 0 if full[0] == 1 else full[1]
    stride_j = 0 if full[1] == 1 else 1
    return stride_i, stride_j


def gemm(A, B, C=None, *, alpha=1.0, beta=1.0, transA=False, transB=False, relu=False,
         want_s=True):
    """ONNX Gemm by its definition, in fp64.  Returns ``(Y, S)``."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    B = np.ascontiguousarray(B, dtype=np.float32)
    if A.ndim != 2 or B.ndim != 2:
        raise OracleShapeError("A and B must be rank 2")
    M, K = (A.shape[1], A.shape[0]) if transA else A.shape
    Kb, N = (B.shape[1], B.shape[0]) if transB else B.shape
    if K != Kb:
        raise OracleShapeError("inner dimensions differ")
    si = sj = 0
    if C is not None:
        C = np.ascontiguousarray(C, dtype=np.float32)
        si, sj = gemm_c_strides(C.shape, M, N)
    Y = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64) if want_s else None
    _load().onnx_oracle_gemm(
        A.ctypes.data, B.ctypes.data, C.ctypes.data if C is not None else None,
        M, N, K, int(bool(transA)), int(bool(transB)), float(alpha), float(beta),
        si, sj, int(bool(relu)), Y.ctypes.data, S.ctypes.data if S is not None else None)
    return Y, S
