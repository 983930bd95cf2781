"""CPU-side checks of the product's host logic: the descriptor layer against the
oracle's independent shape resolver (bit-exact), error codes, and that the shared
library loads and exports every symbol the public header declares."""
import ctypes
import os
import re

import pytest
from hypothesis import given, settings, strategies as st

import oracle
from paper_2008_08272_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    header = open(os.path.join(ROOT, "include", "onnx_b200.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(onnxb?_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS) | (declared - set(binding.EXPORTS))
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared but not exported"
    for name in binding.EXPORTS:
        assert name in declared, f"{name} is bound but not declared in the header"


def test_status_strings_and_launch_counter():
    lib = binding.load()
    seen = {lib.onnxb_status_string(i) for i in range(8)}
    assert len(seen) == 8 and all(s for s in seen)
    assert binding.launch_count() >= 0


AUTO = ["NOTSET", "SAME_UPPER", "SAME_LOWER", "VALID"]

problem = st.fixed_dictionaries(dict(
    N=st.integers(1, 3), Cg=st.integers(1, 5), Mg=st.integers(1, 5), group=st.integers(1, 4),
    H=st.integers(1, 40), W=st.integers(1, 40), kH=st.integers(1, 7), kW=st.integers(1, 7),
    sh=st.integers(1, 4), sw=st.integers(1, 4), dh=st.integers(1, 3), dw=st.integers(1, 3),
    pads=st.tuples(*[st.integers(0, 4)] * 4), auto=st.sampled_from(AUTO),
))


@given(p=problem)
@settings(max_examples=400, deadline=None)
def test_descriptor_matches_oracle_resolver(p):
    x = (p["N"], p["Cg"] * p["group"], p["H"], p["W"])
    w = (p["Mg"] * p["group"], p["Cg"], p["kH"], p["kW"])
    kw = dict(strides=(p["sh"], p["sw"]), dilations=(p["dh"], p["dw"]), group=p["group"], auto_pad=p["auto"])
    pads = p["pads"] if p["auto"] == "NOTSET" else (0, 0, 0, 0)
    try:
        want_y, want_pads = oracle.conv2d_output_shape(x, w, pads=pads, **kw)
    except oracle.OracleShapeError:
        with pytest.raises(binding.OnnxB200Error):
            binding.Conv2dDesc(x, w, pads=pads, **kw)
        return
    d = binding.Conv2dDesc(x, w, pads=pads, **kw)
    assert d.y_shape == tuple(want_y)
    assert d.pads == tuple(want_pads)
    d.close()


def test_descriptor_defaults_and_error_codes():
    d = binding.Conv2dDesc((2, 4, 9, 9), (6, 4, 3, 3))          # every default
    assert d.y_shape == (2, 6, 7, 7) and d.pads == (0, 0, 0, 0)
    d.close()
    d = binding.Conv2dDesc((1, 4, 9, 9), (6, 4, 3, 3), kernel_shape=(3, 3))
    d.close()

    def status(**kw):
        x = kw.pop("x", (1, 4, 9, 9))
        w = kw.pop("w", (4, 4, 3, 3))
        with pytest.raises(binding.OnnxB200Error) as e:
            binding.Conv2dDesc(x, w, **kw)
        return binding.STATUS_NAMES[e.value.status]

    assert status(kernel_shape=(2, 3)) == "ERR_ATTR"
    assert status(strides=(0, 1)) == "ERR_ATTR"
    assert status(strides=(-1, 1)) == "ERR_ATTR"
    assert status(dilations=(1, -2)) == "ERR_ATTR"
    assert status(group=-1) == "ERR_ATTR"
    assert status(auto_pad=9) == "ERR_ATTR"
    assert status(auto_pad="SAME_UPPER", pads=(1, 0, 0, 0)) == "ERR_ATTR"
    assert status(auto_pad="VALID", pads=(0, 0, 0, 1)) == "ERR_ATTR"
    assert status(w=(4, 3, 3, 3)) == "ERR_SHAPE"
    assert status(w=(5, 2, 3, 3), group=2) == "ERR_SHAPE"
    assert status(x=(1, 4, 2, 9)) == "ERR_SHAPE"                 # kernel taller than the input
    assert status(x=(0, 4, 9, 9)) == "ERR_SHAPE"
    assert status(pads=(-1, 0, 0, 0)) == "ERR_UNSUPPORTED"
    assert status(x=(4096, 1024, 1024, 1), w=(1, 1024, 1, 1)) == "ERR_UNSUPPORTED"   # > 2^31-1 elements

    lib = binding.load()
    h = ctypes.c_void_p()
    assert lib.onnx_conv2d_desc(None, ctypes.byref(h)) == 1
    a = binding.make_attrs((1, 4, 9, 9), (4, 4, 3, 3))
    assert lib.onnx_conv2d_desc(ctypes.byref(a), None) == 1
    a.reserved = 1
    assert lib.onnx_conv2d_desc(ctypes.byref(a), ctypes.byref(h)) == 2
    assert lib.onnx_conv2d_desc_query(None, None, None, None) == 1
    assert lib.onnx_conv2d_desc_query_kernel(None) == -1
    lib.onnx_conv2d_desc_destroy(None)                           # must be a no-op


def test_run_calls_reject_bad_arguments_before_any_launch():
    """Argument errors are reported before CUDA is touched, so this runs without a GPU."""
    lib = binding.load()
    before = binding.launch_count()
    d = binding.Conv2dDesc((1, 4, 9, 9), (4, 4, 3, 3), has_bias=True)
    fake = ctypes.c_void_p(0x1000)
    assert lib.onnx_conv2d_run(None, fake, fake, fake, fake, None, 0, None) == 1
    assert lib.onnx_conv2d_run(d._h, None, fake, fake, fake, None, 0, None) == 1
    assert lib.onnx_conv2d_run(d._h, fake, fake, None, fake, None, 0, None) == 1      # bias promised, absent
    assert lib.onnx_conv2d_run(d._h, fake, fake, fake, ctypes.c_void_p(0x1004), None, 0, None) == 4
    d.close()
    d = binding.Conv2dDesc((1, 4, 9, 9), (4, 4, 3, 3))
    assert lib.onnx_conv2d_run(d._h, fake, fake, fake, fake, None, 0, None) == 1      # bias given, not promised
    d.close()
    i64 = ctypes.c_int64
    dims = (i64 * 2)(3, 5)
    g = lambda M, N, K, C=None, rank=0, cd=None, A=fake, Y=fake: lib.onnx_gemm_run(
        0, 0, 1.0, 1.0, M, N, K, A, fake, C, rank, cd, 0, Y, None, 0, None)
    assert g(4, 5, 6, A=None) == 1
    assert g(0, 5, 6) == 3
    assert g(4, 5, 6, C=fake, rank=2, cd=dims) == 3              # (3,5) does not broadcast to (4,5)
    assert g(4, 5, 6, C=fake, rank=1, cd=(i64 * 1)(4)) == 3      # 1-D C of length M is not per-column
    assert g(4, 5, 6, C=fake, rank=3, cd=dims) == 3
    assert g(4, 5, 6, C=fake, rank=1, cd=None) == 1
    assert g(1 << 20, 1 << 20, 4) == 4
    assert g(4, 5, 6, Y=ctypes.c_void_p(0x1008)) == 4
    assert binding.launch_count() == before
