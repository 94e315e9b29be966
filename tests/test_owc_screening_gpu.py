"""The clipping search screens all strengths with a few slice-pair products and forms the accurate loss only
for the strengths within 1 % of a column's smallest screened loss (paper: the grid search over the clipping
strength after Eq. 2).  The screen must never lose the strength the oracle picks from its fp64 loss table:
every column of these layers is compared, on grids whose screen keeps two slices (2, 3 and 4 bits) and on a
finer grid whose screen keeps three (8 bits); a column whose strength differs has to be a near-tie of the
oracle's own table."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs

pytestmark = pytest.mark.gpu

TIE = 1e-7


@pytest.mark.parametrize("base,bits,group,d_in,d_out", [
    ("C2", 2, 128, 2048, 1024),
    ("C4", 3, 128, 2048, 768),
    ("C2", 4, 0, 1536, 512),
    ("C2", 8, 256, 1024, 512),
])
def test_screened_search_picks_the_oracles_strength(base, bits, group, d_in, d_out):
    dev = "cuda:0"
    cfg = inputs.CONFIGS[base].scaled(d_in=d_in, d_out=d_out, n=8192, bits=bits, group_size=group, seed=900 + bits)
    X, W = inputs.make_layer(cfg, device=dev)
    # a few heavy outliers: a clipped weight leaves a residual far above the typical rounding error, which is what the
    # truncating slices of the screen are weakest on
    rng = np.random.default_rng(5)
    rows, cols = rng.integers(0, d_in, 64), rng.integers(0, d_out, 64)
    W[torch.from_numpy(rows).to(dev), torch.from_numpy(cols).to(dev)] *= 6.0
    grid = B.Grid(cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi)
    H = B.cdq_hessian(X)
    scale, zero, Q, gamma = B.cdq_init_rtn(W, grid, H=H)
    init = oracle.init_rtn(W.cpu(), cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi, H=H.cpu().numpy(),
                           want_loss_table=True)
    gg = oracle.gamma_grid(cfg.n_clip, cfg.clip_lo, cfg.clip_hi).astype(np.float32)
    got, want = gamma.cpu().numpy(), gg[init["gamma_idx"]]
    differs = np.nonzero(got != want)[0]
    for j in differs:
        t = init["loss_table"][:, j]
        k = int(np.argmin(np.abs(gg - got[j])))
        gap = abs(t[k] - t[init["gamma_idx"][j]]) / t[init["gamma_idx"][j]]
        assert gap <= TIE, (int(j), float(got[j]), float(want[j]), gap)
    same = got == want
    assert np.array_equal(Q.cpu().numpy()[:, same], init["Q"][:, same])
    assert np.array_equal(scale.cpu().numpy()[:, same], init["scale"][:, same])
    print(f"{bits}-bit g={group} {d_in}x{d_out}: strength differs on {len(differs)} of {d_out} columns (near-ties)")
