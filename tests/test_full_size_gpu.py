"""GPU parity at the full d_in x d_out of the benchmark layers, in the launch configuration
`bench.py` times, checked on sampled columns that the oracle solves one by one.

The oracle cannot form H from the full number of calibration rows in test time, and it does
not have to: H is an input of the descent.  Both sides get the same fp32 H, built here from a
few thousand seeded rows with a library matmul (an input generator, none of the method's
arithmetic) plus a small ridge so that it is positive definite.  The CUDA library then runs
grid + codes, the descent and the loss on ALL columns; the oracle runs the same three steps
on a seeded sample of columns (columns are independent problems: paper, Section 3, Eq. 1).

Bars as in test_parity_gpu.py: every sampled column equals the oracle's codes or forked from the
oracle's trajectory at a step the oracle itself scores as an fp32 near-tie (oracle/audit.py), the summed
column losses within 1e-4 relative; plus properties that hold at any size (budget and convergence
accounting, loss never above the starting loss).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs
from tests.util import compare_pairs_with_oracle, compare_with_oracle, grid_of

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
    return compare_with_oracle(cfg, Hd.cpu().numpy(), Hd, Wd, cols, g, scale, zero, Q0, Q, gamma, per,
                               cfg.passes * cfg.d_in, label=cfg.name)


def test_c1_full_size_sampled_columns():
    _run(inputs.CONFIGS["C1"], rows=8192, n_sample=96)


def test_c2_full_size_owc_sampled_columns():
    _run(inputs.CONFIGS["C2"], rows=16384, n_sample=48)


def test_c3_full_size_sampled_columns():
    _run(inputs.CONFIGS["C3"], rows=16384, n_sample=64)


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
    Qcd = Q.clone()
    stats = B.cdq_bcd_solve(Hd, Wd, g, scale, zero, Q, 2, T, seed=seed)
    loss, per = B.cdq_layer_loss(Hd, Wd, g, scale, zero, Q, per_col=True)
    assert B.load().cdq_last_device_status() == 0
    assert stats["steps"] == T * cfg.d_out and 0 < stats["committed"] < stats["steps"]
    assert stats["loss_after"] < stats["loss_before"]
    np.testing.assert_allclose(stats["loss_after"], loss, rtol=1e-5)

    rng = np.random.default_rng(cfg.seed + 23)
    cols = np.sort(rng.choice(cfg.d_out, 64, replace=False))
    compare_pairs_with_oracle(cfg, Hd.cpu().numpy(), Hd, Wd, cols, g, scale, zero, Qcd, Q, per, T, seed, label="C1")


def test_c4_shaped_full_d_in_sampled_columns():
    """The longest columns of the benchmark layers (d_in = 18432, groups of 128, clipping search): the
    kernel configuration of C4 on 592 of its columns (four per SM), the oracle on 32 of them."""
    _run(inputs.CONFIGS["C4"].scaled(d_out=592), rows=8192, n_sample=32)


def test_c4_shaped_pairs_after_the_greedy_descent_sampled_columns():
    """Pairs on the longest columns (d_in = 18432, groups of 128: the 12-pairs-per-thread configuration),
    from the greedy solution, on 148 columns; the oracle takes the same stages on six of them."""
    cfg = inputs.CONFIGS["C4"].scaled(d_out=148, n_clip=1, clip_lo=1.0, clip_hi=1.0)
    dev = "cuda:0"
    Hd = _h_from_rows(cfg, 8192)
    Wd = inputs.make_w(cfg, device=dev)
    g = grid_of(cfg)
    T, seed = 64, 8
    scale, zero, Q, _ = B.cdq_init_rtn(Wd, g)
    B.cdq_cd_solve(Hd, Wd, g, scale, zero, Q, cfg.passes)
    Qcd = Q.clone()
    stats = B.cdq_bcd_solve(Hd, Wd, g, scale, zero, Q, 2, T, seed=seed)
    loss, per = B.cdq_layer_loss(Hd, Wd, g, scale, zero, Q, per_col=True)
    assert B.load().cdq_last_device_status() == 0
    assert stats["steps"] == T * cfg.d_out and stats["loss_after"] <= stats["loss_before"]
    np.testing.assert_allclose(stats["loss_after"], loss, rtol=1e-5)

    cols = np.array([5, 29, 71, 103, 140, 147])
    compare_pairs_with_oracle(cfg, Hd.cpu().numpy(), Hd, Wd, cols, g, scale, zero, Qcd, Q, per, T, seed, label="C4-shaped",
                              min_same_start=0.5)


def test_mid_size_columns_sampled():
    """Columns between the L2-served and the longest ones (d_in = 6144: two 256-thread teams per SM, rows by one
    bulk copy each), 296 columns, the oracle on 32 of them."""
    _run(inputs.CONFIGS["C3"].scaled(d_in=6144, d_out=296, seed=61), rows=8192, n_sample=32)


def test_rows_of_exactly_48_kb_sampled():
    """d_in = 12288 per-channel: the row takes exactly 48 KB of dynamic shared memory, which together with the
    kernel's static shared memory needs the opt-in for large shared memory (a launch error before it was
    requested for this size too)."""
    _run(inputs.CONFIGS["C3"].scaled(d_in=12288, d_out=148, seed=63), rows=8192, n_sample=16)


def test_ragged_long_columns_sampled():
    """d_in = 11008 (not a multiple of the team's footprint: the last chunk slots reach past the row), rows
    from HBM by one bulk copy, 296 columns, the oracle on 32 of them."""
    _run(inputs.CONFIGS["C3"].scaled(d_in=11008, d_out=296, seed=67), rows=8192, n_sample=32)


def test_long_columns_whose_length_is_not_a_multiple_of_four_sampled():
    """d_in = 6146 (rows of H are then not 16-byte aligned: no bulk copies, the kernel that keeps the row in
    registers runs with scalar loads at the ragged end), 148 columns, the oracle on 32 of them."""
    _run(inputs.CONFIGS["C3"].scaled(d_in=6146, d_out=148, seed=71), rows=8192, n_sample=32)


# Row lengths (in entries) at which the kernel that stages rows through shared memory changes its team shape,
# each with a length just inside the next shape; 12224 and 12288 are the lengths whose row fills the 48 KB of
# shared memory that need no opt-in (together with the kernel's own static shared memory they exceed it).
_SHAPE_EDGES = [4 * c for c in (1024, 2048, 2304, 2560, 2816, 3072, 3328, 3584, 3840, 4096, 4224, 4608)]
ROW_LENGTHS = {
    0: sorted(set([2304, 12224] + _SHAPE_EDGES + [d + 16 for d in _SHAPE_EDGES[:-1]])),
    128: sorted(set([2304, 12160] + _SHAPE_EDGES + [d + 128 for d in _SHAPE_EDGES[:-1]])),
}


@pytest.mark.parametrize("group", [0, 128])
def test_every_team_shape_of_the_long_row_kernel(group):
    """Every team shape of the long-row descent kernel, with a full and with a ragged team: 6 columns, 24 steps
    each, the loss of the result from the descent's gradient; codes, grids and losses against the oracle."""
    dev = "cuda:0"
    for d_in in ROW_LENGTHS[group]:
        cfg = inputs.CONFIGS["C3"].scaled(d_in=d_in, d_out=6, bits=3, group_size=group, n_clip=1, clip_lo=1.0, clip_hi=1.0,
                                          seed=500 + d_in % 97)
        Hd = _h_from_rows(cfg, 512, ridge=1e-2)
        Wd = inputs.make_w(cfg, device=dev)
        g = grid_of(cfg)
        scale, zero, Q0, gamma = B.cdq_init_rtn(Wd, g)
        Q = Q0.clone()
        budget = 24
        stats, loss, per = B.cdq_cd_solve_with_loss(Hd, Wd, g, scale, zero, Q, budget, per_col=True)
        assert B.load().cdq_last_device_status() == 0
        assert stats["committed"] == budget * cfg.d_out, (d_in, stats)
        compare_with_oracle(cfg, Hd.cpu().numpy(), Hd, Wd, np.arange(cfg.d_out), g, scale, zero, Q0, Q, gamma, per, budget,
                            label=f"d_in={d_in} g={group}")


def test_longest_rows_with_small_groups_take_the_cache_served_kernel():
    """d_in = 18432 in groups of 16: row buffer, H_ii tables and 1152 group scales do not fit in one block's shared
    memory together, so the descent runs in the kernel that reads rows and tables through the caches; same bars."""
    dev = "cuda:0"
    cfg = inputs.CONFIGS["C3"].scaled(d_in=18432, d_out=6, bits=3, group_size=16, n_clip=1, clip_lo=1.0, clip_hi=1.0, seed=77)
    Hd = _h_from_rows(cfg, 512, ridge=1e-2)
    Wd = inputs.make_w(cfg, device=dev)
    g = grid_of(cfg)
    scale, zero, Q0, gamma = B.cdq_init_rtn(Wd, g)
    Q = Q0.clone()
    budget = 24
    stats, loss, per = B.cdq_cd_solve_with_loss(Hd, Wd, g, scale, zero, Q, budget, per_col=True)
    assert B.load().cdq_last_device_status() == 0
    assert stats["committed"] == budget * cfg.d_out
    compare_with_oracle(cfg, Hd.cpu().numpy(), Hd, Wd, np.arange(cfg.d_out), g, scale, zero, Q0, Q, gamma, per, budget,
                        label="d_in=18432 g=16")
