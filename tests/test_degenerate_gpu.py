"""Degenerate layers on the GPU against the oracle: a dead input feature (zero row and column of
H), two identical features (a singular 2 x 2 block of H), fewer calibration rows than features
(rank-deficient H), a constant weight column and a constant group (grids with one point).

The fp64 verification mode has to stay bit-exact here too; the production mode has to reach the
oracle's loss, and must never move a coordinate whose grid has one point."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs

pytestmark = pytest.mark.gpu


def _layer(bits, g, seed=91, d_in=64, d_out=12, n=40):
    cfg = inputs.CONFIGS["C0"].scaled(d_in=d_in, d_out=d_out, n=n, bits=bits, group_size=g, passes=2, seed=seed,
                                      n_clip=1, clip_lo=1.0, clip_hi=1.0)
    X, W = inputs.make_layer(cfg)
    X = X.clone(); W = W.clone()
    X[:, 5] = 0.0                      # dead feature
    X[:, 9] = X[:, 8]                  # duplicated feature
    W[:, 3] = 0.0123                   # constant column
    gg = g if g else d_in
    W[gg:2 * gg, 7] = -0.5 if 2 * gg <= d_in else W[gg:2 * gg, 7]   # constant group in column 7 (grouped grids)
    _, H32 = oracle.hessian(X, 0.0)
    init = oracle.init_rtn(W, bits, g, 1, 1.0, 1.0)
    return cfg, X, W, H32, init


def _dev(cfg, W, H32, init):
    dev = "cuda:0"
    return (torch.from_numpy(np.ascontiguousarray(H32)).to(dev), W.to(dev), B.Grid(cfg.bits, cfg.group_size, 1, 1.0, 1.0),
            torch.from_numpy(init["scale"]).to(dev), torch.from_numpy(init["zero"]).to(dev),
            torch.from_numpy(init["Q"]).to(dev).clone())


@pytest.mark.parametrize("bits,g", [(2, 0), (3, 16), (4, 0)])
def test_hessian_grid_and_descent_verify_mode(bits, g):
    cfg, X, W, H32, init = _layer(bits, g)
    Hg = B.cdq_hessian(X.to("cuda:0"), mode="verify")
    assert np.array_equal(Hg.cpu().numpy(), H32)
    assert (H32[5] == 0).all() and (H32[:, 5] == 0).all() and H32[8, 8] == H32[9, 9] == H32[8, 9]
    Hd, Wd, grid, scale, zero, Q = _dev(cfg, W, H32, init)
    s2, z2, Q2, _ = B.cdq_init_rtn(Wd, grid, mode="verify")
    assert np.array_equal(s2.cpu().numpy(), init["scale"]) and np.array_equal(Q2.cpu().numpy(), init["Q"])
    assert (init["scale"][:, 3] == 0).all()                       # the constant column's grid has one point
    ref = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in, g)
    stats = B.cdq_cd_solve(Hd, Wd, grid, scale, zero, Q, cfg.passes, mode="verify")
    assert np.array_equal(Q.cpu().numpy(), ref["Q"])
    assert stats["committed"] == ref["committed"] and stats["columns_converged"] == ref["columns_converged"]
    loss = B.cdq_layer_loss(Hd, Wd, grid, scale, zero, Q, mode="verify")
    np.testing.assert_allclose(loss, oracle.layer_loss(H32, W, init["scale"], init["zero"], ref["Q"], g)[0], rtol=1e-13)


@pytest.mark.parametrize("bits,g", [(2, 0), (3, 16)])
def test_pairs_verify_mode(bits, g):
    cfg, X, W, H32, init = _layer(bits, g, seed=92)
    Hd, Wd, grid, scale, zero, Q = _dev(cfg, W, H32, init)
    ref = oracle.bcd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], 2, 96, seed=4, group_size=g)
    stats = B.cdq_bcd_solve(Hd, Wd, grid, scale, zero, Q, 2, 96, seed=4, mode="verify")
    assert np.array_equal(Q.cpu().numpy(), ref["Q"])
    assert stats["committed"] == int(ref["moves"].sum())


@pytest.mark.parametrize("bits,g", [(2, 0), (3, 16), (4, 0)])
def test_production_mode_reaches_the_oracle_loss(bits, g):
    cfg, X, W, H32, init = _layer(bits, g, seed=93, d_in=256, d_out=40, n=150)
    Hd, Wd, grid, scale, zero, Q = _dev(cfg, W, H32, init)
    ref = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in, g)
    ref_loss = oracle.layer_loss(H32, W, init["scale"], init["zero"], ref["Q"], g)[0]
    B.cdq_cd_solve(Hd, Wd, grid, scale, zero, Q, cfg.passes)
    loss = B.cdq_layer_loss(Hd, Wd, grid, scale, zero, Q)
    assert B.load().cdq_last_device_status() == 0
    got = Q.cpu().numpy()
    # a rank-deficient H has many exactly tied moves, which fp32 scores may order differently:
    # the bar is the loss, and the coordinates that cannot move
    assert abs(loss - ref_loss) <= 1e-3 * ref_loss + 1e-12
    assert np.array_equal(got[:, 3], init["Q"][:, 3])             # constant column: untouched
    assert np.array_equal(got[5], init["Q"][5])                   # dead feature: no move lowers the loss
    Qb = Q.clone()
    refb = oracle.bcd_solve(H32, W, bits, init["scale"], init["zero"], ref["Q"], 2, 64, seed=6, group_size=g)
    B.cdq_bcd_solve(Hd, Wd, grid, scale, zero, Qb, 2, 64, seed=6)
    lb = B.cdq_layer_loss(Hd, Wd, grid, scale, zero, Qb)
    assert lb <= loss * (1 + 1e-9)
    assert abs(lb - refb["loss_after"].sum()) <= 1e-3 * refb["loss_after"].sum() + 1e-12
    assert np.array_equal(Qb.cpu().numpy()[:, 3], init["Q"][:, 3])
