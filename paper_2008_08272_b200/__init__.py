"""ONNX Conv and Gemm for B200 (sm_100a): C-ABI library plus a thin Python binding.

``workloads`` (seeded synthetic inputs) imports without the CUDA library; the
operator entry points are loaded on first use from ``binding`` and raise if the
compiled library is missing - there is no CPU fallback.
"""
from importlib import import_module

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in __all__:
        return import_module(f"{__name__}.{name}")
    raise AttributeError(name)
