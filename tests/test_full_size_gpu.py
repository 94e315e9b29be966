"""GPU parity at the full d_in x d_out of the benchmark layers, in the launch configuration
`bench.py` times, checked on sampled columns that the oracle solves one by one.

The oracle cannot form H from the full number of calibration rows in test time, and it does
not have to: H is an input of the descent.  Both sides get the same fp32 H, built here from a
few thousand seeded rows with a library matmul (an input generator, none of the method's
arithmetic) plus a small ridge so that it is positive definite.  The CUDA library then runs
grid + codes, the descent and the loss on ALL columns; the oracle runs the same three steps
on a seeded sample of columns (columns are independent problems: paper, Section 3, Eq. 1).

Bars as in test_parity_gpu.py: >= 99.9 % equal codes over the sampled columns, loss within
1e-4 relative; plus properties that hold at any size (budget and convergence accounting,
loss never above the starting loss).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs
from tests.util import grid_of

pytestmark = pytest.mark.gpu

CODE_AGREE = 0.999
LOSS_RTOL = 1e-4


def _h_from_rows(cfg, rows, ridge=1e-3):
    X = inputs.make_x(cfg.scaled(n=rows), device="cuda:0").double()
    H = (X.T @ X)
    H += ridge * H.diagonal().mean() * torch.eye(cfg.d_in, dtype=torch.float64, device=H.device)
    return H.float().contiguous()


def _run(cfg, rows, n_sample, owc=True):
    dev = "cuda:0"
    if not owc:
        cfg = cfg.scaled(n_clip=1, clip_lo=1.0, clip_hi=1.0)
    Hd = _h_from_rows(cfg, rows)
    Wd = inputs.make_w(cfg, device=dev)
    g = grid_of(cfg)
    scale, zero, Q0, gamma = B.cdq_init_rtn(Wd, g, H=Hd if cfg.n_clip > 1 else None)
    Q = Q0.clone()
    stats = B.cdq_cd_solve(Hd, Wd, g, scale, zero, Q, cfg.passes)
    loss, per = B.cdq_layer_loss(Hd, Wd, g, scale, zero, Q, per_col=True)
    assert B.load().cdq_last_device_status() == 0

    # properties at any size
    assert stats["steps"] == cfg.passes * cfg.d_in * cfg.d_out
    assert 0 < stats["committed"] <= stats["steps"]
    assert stats["columns_converged"] <= cfg.d_out
    assert stats["loss_after"] <= stats["loss_before"]
    np.testing.assert_allclose(stats["loss_after"], loss, rtol=1e-5)
    assert int(Q.max()) <= (1 << cfg.bits) - 1

    # sampled columns against the oracle
    rng = np.random.default_rng(cfg.seed + 17)
    cols = np.sort(rng.choice(cfg.d_out, n_sample, replace=False))
    H32 = Hd.cpu().numpy()
    Wc = Wd[:, torch.from_numpy(cols).to(dev)].cpu()
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi,
                           H=H32 if cfg.n_clip > 1 else None)
    same = np.ones(n_sample, dtype=bool)
    if cfg.n_clip > 1:
        grid = oracle.gamma_grid(cfg.n_clip, cfg.clip_lo, cfg.clip_hi)
        same = gamma.cpu().numpy()[cols] == grid[init["gamma_idx"]].astype(np.float32)
        assert same.mean() >= 0.95, same.mean()
    keep = np.nonzero(same)[0]
    assert np.array_equal(Q0.cpu().numpy()[:, cols][:, keep], init["Q"][:, keep])
    res = oracle.cd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in,
                          cfg.group_size)
    _, per_ref = oracle.layer_loss(H32, Wc, init["scale"], init["zero"], res["Q"], cfg.group_size)
    got = Q.cpu().numpy()[:, cols]
    agree = float((got[:, keep] == res["Q"][:, keep]).mean())
    assert agree >= CODE_AGREE, agree
    per_got = per.cpu().numpy()[cols]
    assert abs(per_got[keep].sum() - per_ref[keep].sum()) <= LOSS_RTOL * per_ref[keep].sum()
    return agree


def test_c1_full_size_sampled_columns():
    _run(inputs.CONFIGS["C1"], rows=8192, n_sample=96)


def test_c2_full_size_owc_sampled_columns():
    _run(inputs.CONFIGS["C2"], rows=16384, n_sample=48)


def test_c3_full_size_sampled_columns():
    _run(inputs.CONFIGS["C3"], rows=16384, n_sample=6)


def test_c1_full_size_pairs_after_the_greedy_descent_sampled_columns():
    """BCD with random pairs (Algorithm 2) started from the greedy solution, as the paper runs it,
    on all columns of the C1 layer; the oracle takes the same three stages on sampled columns."""
    cfg = inputs.CONFIGS["C1"]
    dev = "cuda:0"
    Hd = _h_from_rows(cfg, 8192)
    Wd = inputs.make_w(cfg, device=dev)
    g = grid_of(cfg)
    T, seed = cfg.d_in // 8, 3
    scale, zero, Q, _ = B.cdq_init_rtn(Wd, g)
    B.cdq_cd_solve(Hd, Wd, g, scale, zero, Q, cfg.passes)
    stats = B.cdq_bcd_solve(Hd, Wd, g, scale, zero, Q, 2, T, seed=seed)
    loss, per = B.cdq_layer_loss(Hd, Wd, g, scale, zero, Q, per_col=True)
    assert B.load().cdq_last_device_status() == 0
    assert stats["steps"] == T * cfg.d_out and 0 < stats["committed"] < stats["steps"]
    assert stats["loss_after"] < stats["loss_before"]
    np.testing.assert_allclose(stats["loss_after"], loss, rtol=1e-5)

    rng = np.random.default_rng(cfg.seed + 23)
    cols = np.sort(rng.choice(cfg.d_out, 64, replace=False))
    H32 = Hd.cpu().numpy()
    Wc = Wd[:, torch.from_numpy(cols).to(dev)].cpu()
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, 1, 1.0, 1.0)
    cd = oracle.cd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in, cfg.group_size)
    ref = oracle.bcd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], cd["Q"], 2, T, seed=seed,
                           group_size=cfg.group_size)
    got = Q.cpu().numpy()[:, cols]
    agree = float((got == ref["Q"]).mean())
    forked = int((got != ref["Q"]).any(axis=0).sum())
    assert agree >= CODE_AGREE or (forked <= 2 and agree >= 0.99), (agree, forked)
    per_got = per.cpu().numpy()[cols]
    assert abs(per_got.sum() - ref["loss_after"].sum()) <= LOSS_RTOL * ref["loss_after"].sum()
    assert ref["moves"].sum() > 0


def test_c4_shaped_full_d_in_sampled_columns():
    """The longest columns of the benchmark layers (d_in = 18432, groups of 128, clipping search): the
    kernel configuration of C4 on 592 of its columns (four per SM), the oracle on four of them."""
    _run(inputs.CONFIGS["C4"].scaled(d_out=592), rows=8192, n_sample=4)


def test_c4_shaped_pairs_after_the_greedy_descent_sampled_columns():
    """Pairs on the longest columns (d_in = 18432, groups of 128: the 12-pairs-per-thread configuration),
    from the greedy solution, on 148 columns; the oracle takes the same stages on three of them."""
    cfg = inputs.CONFIGS["C4"].scaled(d_out=148, n_clip=1, clip_lo=1.0, clip_hi=1.0)
    dev = "cuda:0"
    Hd = _h_from_rows(cfg, 8192)
    Wd = inputs.make_w(cfg, device=dev)
    g = grid_of(cfg)
    T, seed = 64, 8
    scale, zero, Q, _ = B.cdq_init_rtn(Wd, g)
    B.cdq_cd_solve(Hd, Wd, g, scale, zero, Q, cfg.passes)
    stats = B.cdq_bcd_solve(Hd, Wd, g, scale, zero, Q, 2, T, seed=seed)
    loss, per = B.cdq_layer_loss(Hd, Wd, g, scale, zero, Q, per_col=True)
    assert B.load().cdq_last_device_status() == 0
    assert stats["steps"] == T * cfg.d_out and stats["loss_after"] <= stats["loss_before"]
    np.testing.assert_allclose(stats["loss_after"], loss, rtol=1e-5)

    cols = np.array([5, 71, 140])
    H32 = Hd.cpu().numpy()
    Wc = Wd[:, torch.from_numpy(cols).to(dev)].cpu()
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, 1, 1.0, 1.0)
    cd = oracle.cd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in, cfg.group_size)
    ref = oracle.bcd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], cd["Q"], 2, T, seed=seed,
                           group_size=cfg.group_size)
    got = Q.cpu().numpy()[:, cols]
    agree = float((got == ref["Q"]).mean())
    forked = int((got != ref["Q"]).any(axis=0).sum())
    assert agree >= CODE_AGREE or (forked <= 1 and agree >= 0.99), (agree, forked)
    per_got = per.cpu().numpy()[cols]
    assert abs(per_got.sum() - ref["loss_after"].sum()) <= LOSS_RTOL * ref["loss_after"].sum()


def test_mid_size_columns_sampled():
    """Columns between the L2-served and the longest ones (d_in = 6144: two 256-thread teams per SM, rows by one
    bulk copy each), 296 columns, the oracle on six of them."""
    _run(inputs.CONFIGS["C3"].scaled(d_in=6144, d_out=296, seed=61), rows=8192, n_sample=6)


def test_ragged_long_columns_sampled():
    """d_in = 11008 (not a multiple of the team's footprint: the last chunk slots reach past the row), rows
    from HBM by one bulk copy, 296 columns, the oracle on four of them."""
    _run(inputs.CONFIGS["C3"].scaled(d_in=11008, d_out=296, seed=67), rows=8192, n_sample=4)
