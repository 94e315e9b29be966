"""cdq_layer_loss_static: the loss entry point for callers that may not allocate device memory
(its scratch is a fixed array inside the library).  Collected last on purpose, so that a run
that stops at the first failure has already been through every other test.

Checks, through the C ABI: two calls in a row (the shared scratch keeps the first call's
contents) give the same result as cdq_layer_loss with a caller workspace and as the CPU oracle's
loss from the definition (Eq. 1 with H = X^T X), and a layer that does not fit in the fixed array is
refused with a message."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs


def test_oversized_layer_is_refused_before_any_launch():
    lib = B.load()
    import ctypes
    gd = B.Grid(bits=3).c()
    dummy = ctypes.c_void_p(256)   # never dereferenced: the size check comes first
    loss = ctypes.c_double(0.0)
    st = lib.cdq_layer_loss_static(dummy, dummy, 0, 4096, 4096, 4096, ctypes.byref(gd), dummy, dummy, dummy,
                                   ctypes.byref(loss), None, None)
    assert st == 4
    msg = lib.cdq_last_error_detail().decode()
    assert "needs" in msg and str(B.STATIC_SCRATCH_BYTES) in msg


# The workspace version may take the int8 tensor-core path (loss to ~1e-8 relative), the static
# one always runs the fp64 kernels: they agree far inside the 1e-4 bar of the parity tests.
RTOL = 1e-6


@pytest.mark.gpu
def test_static_scratch_matches_workspace_version_twice():
    dev = "cuda:0"
    results = []
    # two different layers back to back: the second call finds the first one's data in the array
    for k, (d_in, d_out, g) in enumerate([(512, 700, 128), (384, 256, 0)]):
        cfg = inputs.CONFIGS["C0"].scaled(d_in=d_in, d_out=d_out, n=2048, bits=3, group_size=g, seed=40 + k)
        X, W = inputs.make_layer(cfg, device=dev)
        grid = B.Grid(cfg.bits, cfg.group_size)
        H = B.cdq_hessian(X)
        scale, zero, Q, _ = B.cdq_init_rtn(W, grid)
        want, want_cols = B.cdq_layer_loss(H, W, grid, scale, zero, Q, per_col=True)
        cols = torch.empty(d_out, dtype=torch.float64, device=dev)
        got = B.cdq_layer_loss_static(H, W, grid, scale, zero, Q, per_col=cols)
        torch.cuda.synchronize()
        results.append((got, want))
        assert abs(got - want) <= RTOL * abs(want)
        np.testing.assert_allclose(cols.cpu().numpy(), want_cols.cpu().numpy(), rtol=RTOL)
        # the expected value itself: the oracle's loss on the same H, W, grid and codes
        ref, ref_cols = oracle.layer_loss(H.cpu().numpy(), W.cpu(), scale.cpu().numpy(), zero.cpu().numpy(),
                                          Q.cpu().numpy(), cfg.group_size)
        assert abs(got - ref) <= RTOL * abs(ref)
        np.testing.assert_allclose(cols.cpu().numpy(), ref_cols, rtol=RTOL)
        # and once more on the same layer, without per-column output
        again = B.cdq_layer_loss_static(H, W, grid, scale, zero, Q)
        assert abs(again - want) <= RTOL * abs(want)
    assert results[0][0] != results[1][0]
