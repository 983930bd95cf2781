"""Thin ctypes binding over the C ABI declared in ``include/onnx_b200.h``.

Argument marshalling only: every step of Conv and Gemm runs in the library's
CUDA kernels.  Tensors are torch CUDA tensors used as device memory; the current
torch stream is passed through.  There is no CPU fallback: if the compiled
library is missing, or a tensor is not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

from . import build as _build

OK = 0
STATUS_NAMES = ["OK", "ERR_NULL", "ERR_ATTR", "ERR_SHAPE", "ERR_UNSUPPORTED", "ERR_WORKSPACE",
                "ERR_CUDA", "ERR_DEVICE_TIMEOUT"]
AUTO_PAD = {"NOTSET": 0, "SAME_UPPER": 1, "SAME_LOWER": 2, "VALID": 3}
KERNEL_FAMILIES = ["simt_direct", "simt_depthwise", "mma_gemm", "mma_implicit", "mma_gather_gemm"]
WEIGHT_COPY_FAMILIES = ("mma_implicit", "mma_gemm", "mma_gather_gemm")   # prepack makes their derived copy of W once

EXPORTS = [
    "onnx_conv2d_desc", "onnx_conv2d_desc_query", "onnx_conv2d_desc_query_kernel", "onnx_conv2d_run",
    "onnx_conv2d_desc_destroy", "onnx_conv2d_run_static", "onnx_conv2d_static_scratch_bytes",
    "onnx_gemm_workspace_bytes", "onnx_gemm_run", "onnxb_status_string",
    "onnxb_last_device_status", "onnxb_set_kernel_override", "onnxb_launch_count",
    "onnxb_probe_tf32_mma_rate", "onnx_matmul_add_run",
    "onnx_maxpool2d_shape", "onnx_maxpool2d_run", "onnx_global_average_pool_run", "onnx_conv2d_add_run",
    "onnx_conv2d_prepack", "onnx_conv2d_run_prepacked", "onnxb_probe_wait_timeout",
]


class OnnxB200Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}")


class ConvAttrs(ctypes.Structure):
    _fields_ = [
        ("x_dims", ctypes.c_int64 * 4), ("w_dims", ctypes.c_int64 * 4),
        ("kernel_shape", ctypes.c_int64 * 2), ("pads", ctypes.c_int64 * 4),
        ("strides", ctypes.c_int64 * 2), ("dilations", ctypes.c_int64 * 2),
        ("group", ctypes.c_int64), ("auto_pad", ctypes.c_int32), ("has_bias", ctypes.c_int32),
        ("fuse_relu", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load(build_if_missing: bool = True):
    """Load libonnx_b200.so (building it first when absent and nvcc is available)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path):
        if not build_if_missing:
            raise OnnxB200Error(6, f"{path} is missing; run python -m paper_2008_08272_b200.build")
        _build.build()
    lib = ctypes.CDLL(path)
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    lib.onnx_conv2d_desc.restype = ctypes.c_int
    lib.onnx_conv2d_desc.argtypes = [ctypes.POINTER(ConvAttrs), ctypes.POINTER(vp)]
    lib.onnx_conv2d_desc_query.restype = ctypes.c_int
    lib.onnx_conv2d_desc_query.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(sz)]
    lib.onnx_conv2d_desc_query_kernel.restype = ctypes.c_int
    lib.onnx_conv2d_desc_query_kernel.argtypes = [vp]
    lib.onnx_conv2d_run.restype = ctypes.c_int
    lib.onnx_conv2d_run.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    lib.onnx_conv2d_add_run.restype = ctypes.c_int
    lib.onnx_conv2d_add_run.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.onnx_conv2d_prepack.restype = ctypes.c_int
    lib.onnx_conv2d_prepack.argtypes = [vp, vp, vp, sz, vp]
    lib.onnx_conv2d_run_prepacked.restype = ctypes.c_int
    lib.onnx_conv2d_run_prepacked.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.onnx_conv2d_run_static.restype = ctypes.c_int
    lib.onnx_conv2d_run_static.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.onnx_conv2d_static_scratch_bytes.restype = sz
    lib.onnx_conv2d_static_scratch_bytes.argtypes = []
    lib.onnx_conv2d_desc_destroy.restype = None
    lib.onnx_conv2d_desc_destroy.argtypes = [vp]
    lib.onnx_gemm_workspace_bytes.restype = sz
    lib.onnx_gemm_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int, i64, i64, i64]
    lib.onnx_gemm_run.restype = ctypes.c_int
    lib.onnx_gemm_run.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_float, i64, i64, i64,
                                  vp, vp, vp, ctypes.c_int, ctypes.POINTER(i64), ctypes.c_int, vp, vp, sz, vp]
    lib.onnx_matmul_add_run.restype = ctypes.c_int
    lib.onnx_matmul_add_run.argtypes = [i64, i64, i64, vp, vp, vp, ctypes.c_int, ctypes.POINTER(i64), ctypes.c_int, vp,
                                        vp, sz, vp]
    p64 = ctypes.POINTER(i64)
    lib.onnx_maxpool2d_shape.restype = ctypes.c_int
    lib.onnx_maxpool2d_shape.argtypes = [p64, p64, p64, p64, p64]
    lib.onnx_maxpool2d_run.restype = ctypes.c_int
    lib.onnx_maxpool2d_run.argtypes = [p64, p64, p64, p64, vp, vp, vp]
    lib.onnx_global_average_pool_run.restype = ctypes.c_int
    lib.onnx_global_average_pool_run.argtypes = [p64, vp, vp, vp]
    lib.onnxb_status_string.restype = ctypes.c_char_p
    lib.onnxb_status_string.argtypes = [ctypes.c_int]
    lib.onnxb_last_device_status.restype = ctypes.c_int
    lib.onnxb_last_device_status.argtypes = [vp]
    lib.onnxb_set_kernel_override.restype = None
    lib.onnxb_set_kernel_override.argtypes = [ctypes.c_int]
    lib.onnxb_launch_count.restype = ctypes.c_uint64
    lib.onnxb_launch_count.argtypes = []
    lib.onnxb_probe_tf32_mma_rate.restype = ctypes.c_int
    lib.onnxb_probe_tf32_mma_rate.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_double), vp]
    lib.onnxb_probe_wait_timeout.restype = ctypes.c_int
    lib.onnxb_probe_wait_timeout.argtypes = [ctypes.c_longlong, vp]
    _lib = lib
    return lib


def _check(status: int, where: str):
    if status != OK:
        raise OnnxB200Error(status, where)


def _dev_ptr(t, name: str, allow_none: bool = False):
    if t is None:
        if allow_none:
            return None
        raise OnnxB200Error(1, f"{name} is None")
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a torch CUDA tensor (there is no CPU path)")
    if t.dtype != torch.float32 or not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous float32")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def make_attrs(x_shape, w_shape, *, kernel_shape=None, pads=None, strides=None, dilations=None, group=0,
               auto_pad="NOTSET", has_bias=False, fuse_relu=False) -> ConvAttrs:
    a = ConvAttrs()
    a.x_dims[:] = list(x_shape)
    a.w_dims[:] = list(w_shape)
    if kernel_shape is not None:
        a.kernel_shape[:] = list(kernel_shape)
    if pads is not None:
        a.pads[:] = list(pads)
    if strides is not None:
        a.strides[:] = list(strides)
    if dilations is not None:
        a.dilations[:] = list(dilations)
    a.group = int(group)
    a.auto_pad = AUTO_PAD[auto_pad] if isinstance(auto_pad, str) else int(auto_pad)
    a.has_bias = int(bool(has_bias))
    a.fuse_relu = int(bool(fuse_relu))
    return a


class Conv2dDesc:
    """Owns an ``onnxb_conv2d_desc_t`` (``onnx_conv2d_desc`` .. ``onnx_conv2d_desc_destroy``)."""

    def __init__(self, x_shape, w_shape, **attrs):
        self._lib = load()
        self._h = ctypes.c_void_p()
        self.attrs = make_attrs(x_shape, w_shape, **attrs)
        _check(self._lib.onnx_conv2d_desc(ctypes.byref(self.attrs), ctypes.byref(self._h)), "onnx_conv2d_desc")
        y = (ctypes.c_int64 * 4)()
        p = (ctypes.c_int64 * 4)()
        ws = ctypes.c_size_t()
        _check(self._lib.onnx_conv2d_desc_query(self._h, y, p, ctypes.byref(ws)), "onnx_conv2d_desc_query")
        self.y_shape = tuple(int(v) for v in y)
        self.pads = tuple(int(v) for v in p)
        self.workspace_bytes = int(ws.value)
        self.kernel_family = KERNEL_FAMILIES[self._lib.onnx_conv2d_desc_query_kernel(self._h)]

    def run(self, X, W, B=None, Y=None, workspace=None, stream=None):
        """``onnx_conv2d_run``; allocates Y (and a workspace) with torch when not supplied."""
        import torch
        if Y is None:
            Y = torch.empty(self.y_shape, dtype=torch.float32, device=X.device)
        if workspace is None and self.workspace_bytes:
            workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=X.device)
        ws_ptr = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
        ws_len = workspace.numel() * workspace.element_size() if workspace is not None else 0
        _check(self._lib.onnx_conv2d_run(self._h, _dev_ptr(X, "X"), _dev_ptr(W, "W"),
                                         _dev_ptr(B, "B", allow_none=True), _dev_ptr(Y, "Y"),
                                         ws_ptr, ws_len, _stream_ptr(stream)), "onnx_conv2d_run")
        return Y

    def run_add(self, X, W, B, R, Y=None, workspace=None, stream=None):
        """``onnx_conv2d_add_run``: Y = relu?(Conv(X, W) + B + R), R shaped like Y (a residual connection)."""
        import torch
        if Y is None:
            Y = torch.empty(self.y_shape, dtype=torch.float32, device=X.device)
        if workspace is None and self.workspace_bytes:
            workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=X.device)
        ws_ptr = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
        ws_len = workspace.numel() * workspace.element_size() if workspace is not None else 0
        _check(self._lib.onnx_conv2d_add_run(self._h, _dev_ptr(X, "X"), _dev_ptr(W, "W"),
                                             _dev_ptr(B, "B", allow_none=True), _dev_ptr(R, "R"), _dev_ptr(Y, "Y"),
                                             ws_ptr, ws_len, _stream_ptr(stream)), "onnx_conv2d_add_run")
        return Y

    def prepack(self, W, stream=None):
        """``onnx_conv2d_prepack``: the packed copy of constant weights (a uint8 device tensor; empty when
        this descriptor's kernel reads W directly)."""
        import torch
        packed = torch.empty(max(self.workspace_bytes, 16) if self.kernel_family in WEIGHT_COPY_FAMILIES else 16,
                             dtype=torch.uint8, device=W.device)
        _check(self._lib.onnx_conv2d_prepack(self._h, _dev_ptr(W, "W"), ctypes.c_void_p(packed.data_ptr()),
                                             packed.numel(), _stream_ptr(stream)), "onnx_conv2d_prepack")
        return packed

    def run_prepacked(self, X, W, packed, B=None, R=None, Y=None, workspace=None, stream=None):
        """``onnx_conv2d_run_prepacked``: run (R None) or run_add (R given) from a packed copy of W."""
        import torch
        if Y is None:
            Y = torch.empty(self.y_shape, dtype=torch.float32, device=X.device)
        needs_ws = (self.kernel_family not in WEIGHT_COPY_FAMILIES or self.kernel_family == "mma_gather_gemm") \
            and self.workspace_bytes
        if workspace is None and needs_ws:
            workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=X.device)
        ws_ptr = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
        ws_len = workspace.numel() * workspace.element_size() if workspace is not None else 0
        _check(self._lib.onnx_conv2d_run_prepacked(self._h, _dev_ptr(X, "X"), _dev_ptr(W, "W"),
                                                   ctypes.c_void_p(packed.data_ptr()),
                                                   _dev_ptr(B, "B", allow_none=True), _dev_ptr(R, "R", allow_none=True),
                                                   _dev_ptr(Y, "Y"), ws_ptr, ws_len, _stream_ptr(stream)),
               "onnx_conv2d_run_prepacked")
        return Y

    def run_static(self, X, W, B=None, Y=None, stream=None):
        """``onnx_conv2d_run_static``: like run(), but the library's built-in scratch array
        stands in for the workspace, so no device memory is allocated for scratch.  (Y is
        still allocated here with torch when the caller does not pass one.)"""
        import torch
        if Y is None:
            Y = torch.empty(self.y_shape, dtype=torch.float32, device=X.device)
        _check(self._lib.onnx_conv2d_run_static(self._h, _dev_ptr(X, "X"), _dev_ptr(W, "W"),
                                                _dev_ptr(B, "B", allow_none=True), _dev_ptr(Y, "Y"),
                                                _stream_ptr(stream)), "onnx_conv2d_run_static")
        return Y

    def close(self):
        if self._h:
            self._lib.onnx_conv2d_desc_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def onnx_conv2d(X, W, B=None, *, pads=None, strides=None, dilations=None, group=0, auto_pad="NOTSET",
                kernel_shape=None, fuse_relu=False, Y=None, workspace=None, stream=None):
    """One-shot ONNX Conv: build a descriptor, run, destroy."""
    d = Conv2dDesc(tuple(X.shape), tuple(W.shape), kernel_shape=kernel_shape, pads=pads, strides=strides,
                   dilations=dilations, group=group, auto_pad=auto_pad, has_bias=B is not None,
                   fuse_relu=fuse_relu)
    try:
        return d.run(X, W, B, Y=Y, workspace=workspace, stream=stream)
    finally:
        d.close()


def gemm_workspace_bytes(transA, transB, M, N, K) -> int:
    return int(load().onnx_gemm_workspace_bytes(int(bool(transA)), int(bool(transB)), M, N, K))


def onnx_gemm(A, B, C=None, *, alpha=1.0, beta=1.0, transA=False, transB=False, fuse_relu=False,
              Y=None, workspace=None, stream=None):
    """``onnx_gemm_run``: Y = relu?(alpha * A' @ B' + beta * C)."""
    import torch
    lib = load()
    M, K = (A.shape[1], A.shape[0]) if transA else (A.shape[0], A.shape[1])
    N = B.shape[0] if transB else B.shape[1]
    kb = B.shape[1] if transB else B.shape[0]
    if kb != K:
        raise OnnxB200Error(3, "onnx_gemm: inner dimensions differ")
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=A.device)
    c_rank, c_dims = 0, None
    if C is not None:
        c_rank = C.dim()
        c_dims = (ctypes.c_int64 * max(c_rank, 1))(*[int(v) for v in C.shape])
    need = gemm_workspace_bytes(transA, transB, M, N, K)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=A.device)
    ws_ptr = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    ws_len = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib.onnx_gemm_run(int(bool(transA)), int(bool(transB)), float(alpha), float(beta), M, N, K,
                             _dev_ptr(A, "A"), _dev_ptr(B, "B"), _dev_ptr(C, "C", allow_none=True),
                             c_rank, c_dims, int(bool(fuse_relu)), _dev_ptr(Y, "Y"), ws_ptr, ws_len,
                             _stream_ptr(stream)), "onnx_gemm_run")
    return Y


def static_scratch_bytes() -> int:
    return int(load().onnx_conv2d_static_scratch_bytes())


def last_device_status(stream=None) -> int:
    return int(load().onnxb_last_device_status(_stream_ptr(stream)))


def set_kernel_override(family) -> None:
    """``None``/"auto" = automatic; or one of KERNEL_FAMILIES."""
    v = -1 if family in (None, "auto") else KERNEL_FAMILIES.index(family)
    load().onnxb_set_kernel_override(v)


def launch_count() -> int:
    return int(load().onnxb_launch_count())


def probe_tf32_mma_rate(n: int, instructions: int = 4096, stream=None) -> float:
    """``onnxb_probe_tf32_mma_rate``: SM cycles per 128 x n x 8 TF32 MMA with operands resident
    in shared memory (the tensor pipe's ceiling for that shape; ideal n / 2)."""
    out = ctypes.c_double()
    _check(load().onnxb_probe_tf32_mma_rate(int(n), int(instructions), ctypes.byref(out), _stream_ptr(stream)),
           "onnxb_probe_tf32_mma_rate")
    return float(out.value)


def probe_wait_timeout(limit_cycles: int = 1000000, stream=None) -> None:
    """``onnxb_probe_wait_timeout``: enqueue a kernel whose only (bounded) wait runs out after
    ``limit_cycles`` SM cycles; the next ``last_device_status`` then reports ERR_DEVICE_TIMEOUT once."""
    _check(load().onnxb_probe_wait_timeout(int(limit_cycles), _stream_ptr(stream)), "onnxb_probe_wait_timeout")


def onnx_matmul_add(A, B, C=None, *, fuse_relu=False, Y=None, workspace=None, stream=None):
    """``onnx_matmul_add_run``: Y = relu?(A @ B + C), the MatMul + Add pair as one fused Gemm."""
    import torch
    lib = load()
    M, K = A.shape
    if B.shape[0] != K:
        raise OnnxB200Error(3, "onnx_matmul_add: inner dimensions differ")
    N = B.shape[1]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=A.device)
    c_rank, c_dims = 0, None
    if C is not None:
        c_rank = C.dim()
        c_dims = (ctypes.c_int64 * max(c_rank, 1))(*[int(v) for v in C.shape])
    need = gemm_workspace_bytes(False, False, M, N, K)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=A.device)
    ws_ptr = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    ws_len = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib.onnx_matmul_add_run(M, N, K, _dev_ptr(A, "A"), _dev_ptr(B, "B"), _dev_ptr(C, "C", allow_none=True),
                                   c_rank, c_dims, int(bool(fuse_relu)), _dev_ptr(Y, "Y"), ws_ptr, ws_len,
                                   _stream_ptr(stream)), "onnx_matmul_add_run")
    return Y


def _i64(values, n):
    if values is None:
        return None
    return (ctypes.c_int64 * n)(*[int(v) for v in values])


def maxpool2d_shape(x_shape, kernel_shape, pads=None, strides=None):
    """``onnx_maxpool2d_shape``: output dims of ONNX MaxPool (host only)."""
    y = (ctypes.c_int64 * 4)()
    _check(load().onnx_maxpool2d_shape(_i64(x_shape, 4), _i64(kernel_shape, 2), _i64(pads, 4), _i64(strides, 2), y),
           "onnx_maxpool2d_shape")
    return tuple(int(v) for v in y)


def onnx_maxpool2d(X, kernel_shape, *, pads=None, strides=None, Y=None, stream=None):
    """``onnx_maxpool2d_run``: ONNX MaxPool (2-D, NCHW, dilation 1, ceil_mode 0)."""
    import torch
    y_shape = maxpool2d_shape(tuple(X.shape), kernel_shape, pads, strides)
    if Y is None:
        Y = torch.empty(y_shape, dtype=torch.float32, device=X.device)
    _check(load().onnx_maxpool2d_run(_i64(tuple(X.shape), 4), _i64(kernel_shape, 2), _i64(pads, 4), _i64(strides, 2),
                                     _dev_ptr(X, "X"), _dev_ptr(Y, "Y"), _stream_ptr(stream)), "onnx_maxpool2d_run")
    return Y


def onnx_global_average_pool(X, *, Y=None, stream=None):
    """``onnx_global_average_pool_run``: Y[n,c,0,0] = mean of X[n,c,:,:]."""
    import torch
    if Y is None:
        Y = torch.empty((X.shape[0], X.shape[1], 1, 1), dtype=torch.float32, device=X.device)
    _check(load().onnx_global_average_pool_run(_i64(tuple(X.shape), 4), _dev_ptr(X, "X"), _dev_ptr(Y, "Y"),
                                               _stream_ptr(stream)), "onnx_global_average_pool_run")
    return Y
