"""cdq_cd_solve_with_loss: the loss of the descent's result taken from the descent's own final gradient
(1/2 sum_i e_i g_i with g = 2 H e) against the loss from its definition (Eq. 1 with H = X^T X): the CPU oracle's
e^T H e on the codes the call returned, and cdq_layer_loss (the product H E) through the C ABI.

The shapes cover both register-resident kernels (rows read directly, rows staged through shared memory), the
per-channel form that runs in code units and the grouped forms, a row length that is not a multiple of 4, a
budget that ends the descent in mid-flight and one that lets every column converge, constant columns (their
grid has one point), and the two fall-backs (the fp64 verification mode; a group size the fast kernels do not
take), which must give the same number by running the definition."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs

pytestmark = pytest.mark.gpu

# (d_in, d_out, group, bits, steps per column, mode)
CASES = [
    (256, 96, 0, 3, 256, "fast"),        # small per-channel layer
    (512, 70, 128, 2, 100, "fast"),      # grouped, budget ends the descent early
    (384, 64, 32, 4, 4 * 384, "fast"),   # grouped, long budget: columns converge
    (1022, 40, 0, 3, 300, "fast"),       # d_in not a multiple of 4
    (4608, 48, 0, 3, 600, "fast"),       # rows staged through shared memory, per-channel
    (6144, 40, 128, 2, 400, "fast"),     # rows staged through shared memory, grouped
    (516, 33, 6, 3, 200, "fast"),        # group size the fast kernels do not take: loss from the definition
    (256, 48, 64, 3, 256, "verify"),     # verification mode: loss from the definition
]


@pytest.mark.parametrize("d_in,d_out,g,bits,steps,mode", CASES)
def test_loss_of_result_matches_definition(d_in, d_out, g, bits, steps, mode):
    dev = "cuda:0"
    cfg = inputs.CONFIGS["C0"].scaled(d_in=d_in, d_out=d_out, n=max(2048, d_in + 512), bits=bits, group_size=g, seed=77)
    X, W = inputs.make_layer(cfg, device=dev)
    if g == 0:
        W[:, 5] = 0.25          # a constant column: one grid point, nothing moves, loss from the start gradient
    grid = B.Grid(bits, g)
    H = B.cdq_hessian(X, mode=mode)
    scale, zero, Q, _ = B.cdq_init_rtn(W, grid, mode=mode)
    Q_ref = Q.clone()
    stats, loss, cols = B.cdq_cd_solve_with_loss(H, W, grid, scale, zero, Q, steps, mode=mode, per_col=True)
    # the same descent without the loss gives the same codes
    B.cdq_cd_solve(H, W, grid, scale, zero, Q_ref, 0, mode=mode, steps_per_col=steps)
    assert torch.equal(Q, Q_ref)
    want, want_cols = oracle.layer_loss(H.cpu().numpy(), W.cpu(), scale.cpu().numpy(), zero.cpu().numpy(), Q.cpu().numpy(), g)
    got_cols = cols.cpu().numpy()
    scale_cols = np.maximum(np.abs(want_cols), 1e-12 * abs(want))
    assert np.max(np.abs(got_cols - want_cols) / scale_cols) <= 1e-9, np.max(np.abs(got_cols - want_cols) / scale_cols)
    assert abs(loss - want) <= 1e-10 * abs(want)
    lib_loss, lib_cols = B.cdq_layer_loss(H, W, grid, scale, zero, Q, mode=mode, per_col=True)
    assert abs(loss - lib_loss) <= 1e-9 * abs(lib_loss)
    # bookkeeping of the descent (start loss plus the fp32 decreases of its moves) tells the same story
    assert abs(stats["loss_after"] - want) <= 1e-4 * abs(want)
    assert stats["committed"] > 0


def test_loss_only_output_and_argument_check():
    import ctypes
    dev = "cuda:0"
    cfg = inputs.CONFIGS["C0"].scaled(d_in=256, d_out=64, n=1024, seed=5)
    X, W = inputs.make_layer(cfg, device=dev)
    grid = B.Grid(cfg.bits, cfg.group_size)
    H = B.cdq_hessian(X)
    scale, zero, Q, _ = B.cdq_init_rtn(W, grid)
    stats, loss = B.cdq_cd_solve_with_loss(H, W, grid, scale, zero, Q, 128)
    want, _ = oracle.layer_loss(H.cpu().numpy(), W.cpu(), scale.cpu().numpy(), zero.cpu().numpy(), Q.cpu().numpy(),
                                cfg.group_size)
    assert abs(loss - want) <= 1e-10 * abs(want)
    # neither output asked for: refused before anything runs
    gd = grid.c()
    st = B.load().cdq_cd_solve_with_loss(H.data_ptr(), W.data_ptr(), 0, 256, 64, 64, ctypes.byref(gd), scale.data_ptr(),
                                        zero.data_ptr(), Q.data_ptr(), 16, 0, None, None, None, None, 0, None)
    assert st == 1
