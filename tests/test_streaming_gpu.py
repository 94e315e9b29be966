"""binding.quantize_layers: layers streamed from pinned host memory, the next layer's upload in flight while the
current one computes.  Every layer must come out exactly as from quantize_layer on its own (same codes, scales,
zeros, loss), whatever the order and mix of shapes, and against the CPU oracle for one of them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs

pytestmark = pytest.mark.gpu


def test_streamed_layers_equal_single_layer_calls():
    shapes = [(512, 96, 4096), (256, 200, 2048), (512, 96, 4096), (1024, 64, 3072), (256, 200, 2048)]
    grid = B.Grid(3, 0)
    layers, single = [], []
    for k, (d_in, d_out, n) in enumerate(shapes):
        cfg = inputs.CONFIGS["C0"].scaled(d_in=d_in, d_out=d_out, n=n, bits=3, group_size=0, seed=300 + k)
        X, W = inputs.make_layer(cfg)
        layers.append((X.pin_memory(), W.pin_memory()))
        out = B.quantize_layer(layers[-1][0], layers[-1][1], grid, 1)
        single.append({k2: (out[k2].clone() if torch.is_tensor(out[k2]) else out[k2]) for k2 in ("Q", "scale", "zero", "loss")})
    bufs: dict = {}
    n_seen = 0
    for k, out in enumerate(B.quantize_layers(iter(layers), grid, 1, host_buffers=bufs)):
        assert not out["Q"].is_cuda and out["Q"].is_pinned()
        assert torch.equal(out["Q"], single[k]["Q"]), k
        assert torch.equal(out["scale"], single[k]["scale"]) and torch.equal(out["zero"], single[k]["zero"])
        assert out["loss"] == single[k]["loss"]
        n_seen += 1
    assert n_seen == len(shapes)
    assert len(bufs) == 3 * 3    # three shapes, three result tensors each: host buffers are reused per shape
    # one layer against the oracle, end to end
    X, W = layers[3]
    _, H32 = oracle.hessian(X)
    init = oracle.init_rtn(W, 3, 0)
    ref = oracle.cd_solve(H32, W, 3, init["scale"], init["zero"], init["Q"], W.shape[0])
    assert float((single[3]["Q"].numpy() == ref["Q"]).mean()) >= 0.999


def test_empty_iterable_yields_nothing():
    assert list(B.quantize_layers(iter([]), B.Grid(3, 0), 1)) == []
