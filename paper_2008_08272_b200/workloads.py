"""Seeded synthetic workloads shaped like the paper's MNIST and ResNet-50 models.

The paper runs the ONNX Model Zoo MNIST and ResNet50 models on their bundled
test data (Sec. 4.2).  Neither the models nor the data are available offline,
so every tensor here is synthetic: the layer shapes of those models, inputs in a
post-Relu-like range, He-normal weights.  This module only draws random numbers
and lists shapes; it contains none of the operators' arithmetic, so both the
CUDA path's tests and the CPU oracle's tests may use it.

Seeds: ``20080827 + 1000 * config + layer_index``; tensors are drawn from one
``numpy.random.default_rng(seed)`` stream in the order X, W, B (A, B, C for Gemm).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np

SEED_BASE = 20080827


@dataclass(frozen=True)
class ConvCase:
    """One ONNX Conv problem: shapes, attributes, value distributions, seed."""
    name: str
    x_shape: Tuple[int, int, int, int]
    w_shape: Tuple[int, int, int, int]
    pads: Tuple[int, int, int, int] = (0, 0, 0, 0)
    strides: Tuple[int, int] = (1, 1)
    dilations: Tuple[int, int] = (1, 1)
    group: int = 1
    has_bias: bool = True
    relu: bool = True
    seed: int = SEED_BASE
    x_dist: str = "uniform01"        # "uniform01" | "uniform11" | "normal"
    w_dist: str = "he_normal"        # "he_normal" | "uniform11" | "normal"
    b_dist: str = "normal001"        # "normal001" | "uniform11" | "normal"

    @property
    def y_shape(self):
        n, _, h, w = self.x_shape
        m, _, kh, kw = self.w_shape
        p = (h + self.pads[0] + self.pads[2] - ((kh - 1) * self.dilations[0] + 1)) // self.strides[0] + 1
        q = (w + self.pads[1] + self.pads[3] - ((kw - 1) * self.dilations[1] + 1)) // self.strides[1] + 1
        return (n, m, p, q)

    @property
    def flops(self) -> int:
        """2 * outputs * (C/g * kH * kW); padded taps counted, the usual convention."""
        n, m, p, q = self.y_shape
        return 2 * n * m * p * q * self.w_shape[1] * self.w_shape[2] * self.w_shape[3]

    @property
    def algorithmic_bytes(self) -> int:
        """4 * (|X read| + |W| + |B| + |Y|); a 1x1 kernel with stride s touches only every
        s-th input row and column, and whole skipped rows need not leave HBM."""
        x = int(np.prod(self.x_shape))
        if self.w_shape[2] == 1 and self.w_shape[3] == 1 and self.strides[0] > 1 and self.pads == (0, 0, 0, 0):
            n, c, h, w = self.x_shape
            x = n * c * ((h + self.strides[0] - 1) // self.strides[0]) * w
        y = int(np.prod(self.y_shape))
        wt = int(np.prod(self.w_shape))
        b = self.w_shape[0] if self.has_bias else 0
        return 4 * (x + wt + b + y)


@dataclass(frozen=True)
class GemmCase:
    """One ONNX Gemm problem.  a_shape / b_shape are the stored (untransposed) shapes."""
    name: str
    a_shape: Tuple[int, int]
    b_shape: Tuple[int, int]
    c_shape: Optional[Tuple[int, ...]] = None
    transA: bool = False
    transB: bool = False
    alpha: float = 1.0
    beta: float = 1.0
    relu: bool = False
    seed: int = SEED_BASE

    @property
    def mnk(self):
        m, k = (self.a_shape[1], self.a_shape[0]) if self.transA else self.a_shape
        n = self.b_shape[0] if self.transB else self.b_shape[1]
        return m, n, k

    @property
    def flops(self) -> int:
        m, n, k = self.mnk
        return 2 * m * n * k


def _draw(rng, shape, dist, fan_in=1):
    if dist == "uniform01":
        return rng.random(shape, dtype=np.float32)
    if dist == "uniform11":
        return (rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)).astype(np.float32)
    if dist == "normal":
        return rng.standard_normal(shape, dtype=np.float32)
    if dist == "normal001":
        return rng.standard_normal(shape, dtype=np.float32) * np.float32(0.01)
    if dist == "he_normal":
        return rng.standard_normal(shape, dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
    raise ValueError(dist)


def conv_inputs(case: ConvCase, images: Optional[int] = None):
    """(X, W, B) as float32 numpy arrays.  ``images`` draws only the first images of X
    (the stream is drawn in X, W, B order, so W and B then differ from the full draw;
    use ``conv_inputs(case)`` and slice when the same weights are needed)."""
    rng = np.random.default_rng(case.seed)
    xs = case.x_shape if images is None else (images,) + tuple(case.x_shape[1:])
    X = _draw(rng, xs, case.x_dist)
    fan_in = case.w_shape[1] * case.w_shape[2] * case.w_shape[3]
    W = _draw(rng, case.w_shape, case.w_dist, fan_in)
    B = _draw(rng, (case.w_shape[0],), case.b_dist) if case.has_bias else None
    return X, W, B


def gemm_inputs(case: GemmCase):
    rng = np.random.default_rng(case.seed)
    A = rng.standard_normal(case.a_shape, dtype=np.float32)
    B = rng.standard_normal(case.b_shape, dtype=np.float32)
    C = rng.standard_normal(case.c_shape, dtype=np.float32) if case.c_shape is not None else None
    return A, B, C


# ---------------------------------------------------------------------------
# The five configurations
# ---------------------------------------------------------------------------

def config1_mnist_conv() -> ConvCase:
    """MNIST-shaped first convolution: 1 -> 8 channels, 5x5, pad 2, then Relu."""
    return ConvCase("cfg1_mnist_conv5x5", (1, 1, 28, 28), (8, 1, 5, 5), pads=(2, 2, 2, 2),
                    seed=SEED_BASE + 1000 * 1, x_dist="uniform11", w_dist="uniform11",
                    b_dist="uniform11", relu=True)


def config2_gemm_head() -> GemmCase:
    """Classifier head: A[64,256] x B[10,256]^T + C[10]."""
    return GemmCase("cfg2_gemm_head", (64, 256), (10, 256), (10,), transB=True,
                    seed=SEED_BASE + 1000 * 2)


def config3_stage2_3x3(batch: int = 32) -> ConvCase:
    return ConvCase("cfg3_res2_3x3", (batch, 64, 56, 56), (64, 64, 3, 3), pads=(1, 1, 1, 1),
                    seed=SEED_BASE + 1000 * 3)


def config4_stem_and_projection(batch: int = 32) -> List[ConvCase]:
    return [
        ConvCase("cfg4a_stem_7x7_s2", (batch, 3, 224, 224), (64, 3, 7, 7), pads=(3, 3, 3, 3),
                 strides=(2, 2), seed=SEED_BASE + 1000 * 4 + 0),
        ConvCase("cfg4b_proj_1x1_s2", (batch, 256, 56, 56), (512, 256, 1, 1), strides=(2, 2),
                 seed=SEED_BASE + 1000 * 4 + 1),
    ]


def resnet50_v1_convs(batch: int = 64, config: int = 5) -> List[ConvCase]:
    """All 53 convolutions of ResNet-50 v1 in execution order.

    v1 places the stride of a down-sampling block on its first 1x1 and on the 1x1
    projection: 1 stem + 16 blocks x 3 + 4 projections = 53 convolutions.
    """
    cases: List[ConvCase] = []

    def add(tag, c, hw, m, k, s, p):
        idx = len(cases)
        cases.append(ConvCase(f"r50_{idx:02d}_{tag}", (batch, c, hw, hw), (m, c, k, k),
                              pads=(p, p, p, p), strides=(s, s),
                              seed=SEED_BASE + 1000 * config + idx))

    add("stem7x7s2", 3, 224, 64, 7, 2, 3)
    blocks = (3, 4, 6, 3)
    cin, hw = 64, 56
    for stage, nblocks in enumerate(blocks):
        mid, out = 64 << stage, 256 << stage
        for b in range(nblocks):
            s = 2 if (b == 0 and stage > 0) else 1
            t = f"s{stage + 2}b{b}"
            add(t + "_1x1a", cin, hw, mid, 1, s, 0)
            hw_out = hw // s
            add(t + "_3x3", mid, hw_out, mid, 3, 1, 1)
            add(t + "_1x1b", mid, hw_out, out, 1, 1, 0)
            if b == 0:
                add(t + "_proj", cin, hw, out, 1, s, 0)
            cin, hw = out, hw_out
    assert len(cases) == 53
    return cases


def config5_depthwise(batch: int = 64) -> ConvCase:
    return ConvCase("cfg5_depthwise_3x3", (batch, 256, 28, 28), (256, 1, 3, 3), pads=(1, 1, 1, 1),
                    group=256, seed=SEED_BASE + 1000 * 5 + 53)


def with_batch(case: ConvCase, batch: int) -> ConvCase:
    return replace(case, x_shape=(batch,) + tuple(case.x_shape[1:]))
