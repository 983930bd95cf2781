"""The chained ResNet-50 run: every operator of the chain is checked against the oracle ON THE
INPUTS THE CHAIN GAVE IT (the device tensors feeding that operator), so a wrong wiring of buffers,
shortcuts or strides fails here even though errors of earlier layers do not accumulate into the
comparison.  Batch 1 at the model's real 224 x 224 size."""
import numpy as np
import pytest

import oracle

from parity import worst_ratio

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def test_graph_is_resnet50_v1():
    from paper_2008_08272_b200.resnet50_chain import build_graph
    ops = build_graph(2)
    kinds = [o.kind for o in ops]
    assert kinds.count("conv") + kinds.count("conv_add") == 53 and kinds.count("conv_add") == 16
    assert kinds[1] == "maxpool" and kinds[-2:] == ["gap", "gemm"]
    # every shortcut is the block's input, or the projection of it in the four down-sampling blocks
    assert sum(1 for o in ops if o.kind == "conv_add" and o.res.endswith("_sc")) == 4


def test_every_operator_of_the_chain_matches_the_oracle():
    from paper_2008_08272_b200 import binding
    from paper_2008_08272_b200.resnet50_chain import Resnet50Chain
    binding.load(build_if_missing=False)
    dev = torch.device("cuda:0")
    net = Resnet50Chain(1, dev)
    rng = np.random.default_rng(224)
    x = torch.from_numpy(rng.random((1, 3, 224, 224), dtype=np.float32)).to(dev)
    logits = net.forward(x)
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    host = {k: v.cpu().numpy() for k, v in net.buf.items()}
    assert np.isfinite(host["logits"]).all() and np.abs(host["logits"]).max() > 0
    worst = 0.0
    for op in net.ops:
        got, src = host[op.dst], host[op.src]
        if op.case is not None:
            W, B = (t.cpu().numpy() for t in net.params[op.name])
            c = op.case
            conv, S = oracle.conv2d(src, W, B, relu=False, pads=c.pads, strides=c.strides)
            want = conv + host[op.res].astype(np.float64) if op.kind == "conv_add" else conv
            if op.relu:
                want = np.maximum(want, 0.0)
            r = worst_ratio(got, want, S)
            assert r <= 1.0, (op.name, r)
            worst = max(worst, r)
        elif op.kind == "maxpool":
            assert np.array_equal(got, oracle.maxpool2d(src, (3, 3), (1, 1, 1, 1), (2, 2))), op.name
        elif op.kind == "gap":
            want, S = oracle.global_average_pool(src)
            assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-5 * S + 1e-7)
        else:
            W, B = (t.cpu().numpy() for t in net.params["fc"])
            want, S = oracle.gemm(src.reshape(1, 2048), W, B)
            assert worst_ratio(got, want, S) <= 1.0
    net.close()
    print("worst err/tol over the 53 convolutions of the chain:", round(worst, 3))
