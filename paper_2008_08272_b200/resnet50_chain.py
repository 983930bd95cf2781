"""ResNet-50 v1 as one chained run of the library's operators (Sec. 4.2 times this model end to end).

The graph is the ONNX Model Zoo ResNet50 with batch normalisation folded into the convolutions (as
an inference compiler's constant propagation leaves it, Sec. 3.4.4): stem Conv 7x7/2 + Relu,
MaxPool 3x3/2, sixteen bottleneck blocks (1x1 -> 3x3 -> 1x1, stride on the first 1x1 of a
down-sampling block and on its 1x1 projection), each closed by Add + Relu fused into the last 1x1
convolution, GlobalAveragePool, Gemm 2048 -> 1000.  Weights are synthetic (He-normal, seeded): the
model file is not available offline.  Only marshalling and buffer bookkeeping happen here; every
operator runs in the library's kernels.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np

from . import binding
from . import workloads as wl


@dataclass
class Op:
    kind: str                 # "conv" | "conv_add" | "maxpool" | "gap" | "gemm"
    name: str
    src: str                  # name of the input tensor
    dst: str                  # name of the output tensor
    res: Optional[str] = None  # residual addend (conv_add)
    case: Optional[wl.ConvCase] = None
    relu: bool = False


def build_graph(batch: int) -> List[Op]:
    """The operator list in execution order, wired by tensor names."""
    convs = wl.resnet50_v1_convs(batch)
    ops: List[Op] = [Op("conv", convs[0].name, "input", "stem", case=convs[0], relu=True),
                     Op("maxpool", "pool1", "stem", "pool1")]
    cur, i = "pool1", 1
    while i < len(convs):
        a, b3, c1 = convs[i], convs[i + 1], convs[i + 2]
        has_proj = i + 3 < len(convs) and convs[i + 3].name.endswith("_proj")
        blk = a.name[:-5]                                  # e.g. r50_01_s2b0
        ops.append(Op("conv", a.name, cur, blk + "_a", case=a, relu=True))
        ops.append(Op("conv", b3.name, blk + "_a", blk + "_b", case=b3, relu=True))
        shortcut = cur
        if has_proj:
            pj = convs[i + 3]
            ops.append(Op("conv", pj.name, cur, blk + "_sc", case=pj, relu=False))
            shortcut = blk + "_sc"
        ops.append(Op("conv_add", c1.name, blk + "_b", blk + "_out", res=shortcut, case=c1, relu=True))
        cur = blk + "_out"
        i += 4 if has_proj else 3
    ops.append(Op("gap", "gap", cur, "pooled"))
    ops.append(Op("gemm", "fc", "pooled", "logits"))
    return ops


class Resnet50Chain:
    def __init__(self, batch: int, device, seed: int = wl.SEED_BASE + 9000, prepack: bool = True):
        import torch
        self.torch = torch
        self.batch, self.dev = batch, device
        self.ops = build_graph(batch)
        rng = np.random.default_rng(seed)
        self.prepack = prepack                  # weights are constants of the graph: pack them once (Sec. 3.4.4)
        self.packed: Dict[str, object] = {}
        self.params: Dict[str, tuple] = {}
        self.descs: Dict[str, binding.Conv2dDesc] = {}
        ws_bytes = 16
        for op in self.ops:
            if op.case is not None:
                c = op.case
                fan = c.w_shape[1] * c.w_shape[2] * c.w_shape[3]
                W = (rng.standard_normal(c.w_shape, dtype=np.float32) * np.float32(np.sqrt(2.0 / fan)))
                if op.kind == "conv_add":
                    W *= np.float32(0.5)                   # keeps the activations of 16 stacked blocks in range
                B = rng.standard_normal((c.w_shape[0],), dtype=np.float32) * np.float32(0.01)
                self.params[op.name] = (torch.from_numpy(W).to(device), torch.from_numpy(B).to(device))
                d = binding.Conv2dDesc(c.x_shape, c.w_shape, pads=c.pads, strides=c.strides, has_bias=True,
                                       fuse_relu=op.relu)
                self.descs[op.name] = d
                ws_bytes = max(ws_bytes, d.workspace_bytes)
                if prepack:
                    self.packed[op.name] = d.prepack(self.params[op.name][0])
        Wf = rng.standard_normal((2048, 1000), dtype=np.float32) * np.float32(np.sqrt(1.0 / 2048))
        Bf = rng.standard_normal((1000,), dtype=np.float32) * np.float32(0.01)
        self.params["fc"] = (torch.from_numpy(Wf).to(device), torch.from_numpy(Bf).to(device))
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        self.fc_workspace = torch.empty(max(binding.gemm_workspace_bytes(False, False, batch, 1000, 2048), 16),
                                        dtype=torch.uint8, device=device)
        # one buffer per tensor of the graph
        self.buf: Dict[str, "torch.Tensor"] = {}
        for op in self.ops:
            if op.case is not None:
                shape = self.descs[op.name].y_shape
            elif op.kind == "maxpool":
                shape = binding.maxpool2d_shape(tuple(self.buf[op.src].shape), (3, 3), (1, 1, 1, 1), (2, 2))
            elif op.kind == "gap":
                s = self.buf[op.src].shape
                shape = (s[0], s[1], 1, 1)
            else:
                shape = (batch, 1000)
            self.buf[op.dst] = torch.empty(shape, dtype=torch.float32, device=device)
        self.flops = sum(op.case.flops for op in self.ops if op.case is not None) + 2 * batch * 2048 * 1000

    def forward(self, x):
        """Enqueue the whole model on the current stream; returns the logits buffer."""
        self.buf["input"] = x
        for op in self.ops:
            src, dst = self.buf[op.src], self.buf[op.dst]
            if op.kind in ("conv", "conv_add") and self.prepack:
                W, B = self.params[op.name]
                R = self.buf[op.res] if op.kind == "conv_add" else None
                self.descs[op.name].run_prepacked(src, W, self.packed[op.name], B, R, Y=dst, workspace=self.workspace)
            elif op.kind == "conv":
                W, B = self.params[op.name]
                self.descs[op.name].run(src, W, B, Y=dst, workspace=self.workspace)
            elif op.kind == "conv_add":
                W, B = self.params[op.name]
                self.descs[op.name].run_add(src, W, B, self.buf[op.res], Y=dst, workspace=self.workspace)
            elif op.kind == "maxpool":
                binding.onnx_maxpool2d(src, (3, 3), pads=(1, 1, 1, 1), strides=(2, 2), Y=dst)
            elif op.kind == "gap":
                binding.onnx_global_average_pool(src, Y=dst)
            else:
                W, B = self.params["fc"]
                binding.onnx_matmul_add(src.view(self.batch, 2048), W, B, Y=dst, workspace=self.fc_workspace)
        return self.buf["logits"]

    def close(self):
        for d in self.descs.values():
            d.close()
        self.descs.clear()
