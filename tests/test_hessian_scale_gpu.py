"""The tensor-core Hessian at the sizes of the benchmark layers (paper: H = X^T X, Section 3 "Notation" and the first
step of Algorithm 1), against the fp64 oracle on sampled entries.

The oracle cannot form a 14336^2 or 18432^2 Hessian from 131072 or 262144 rows in test time, and need not: an entry
H[i, j] depends on feature columns i and j of X only.  The test gathers a few dozen feature columns (tile edges
of the 128 x 256 output tiles, the first and last tile row, random ones), hands that slim matrix to
oracle.hessian_entries and compares every pair among them -- a few thousand entries, diagonal included -- with the
library's H formed from the whole X.  Bar: 1e-4 of sqrt(H_ii H_jj) (fp32 accumulation over up to 262144 rows; the
target for H is 1e-3 relative Frobenius error)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs

pytestmark = pytest.mark.gpu


def _features(d_in, rng, extra=36):
    edges = [0, 1, 63, 64, 127, 128, 129, 255, 256, 257, 383, 384, 511, 512, d_in - 257, d_in - 256, d_in - 129, d_in - 128,
             d_in - 2, d_in - 1, d_in // 2, d_in // 2 + 127, d_in // 2 + 128]
    f = np.unique(np.concatenate([np.array([e for e in edges if 0 <= e < d_in]), rng.integers(0, d_in, extra)]))
    return f


def _check(X, H, label, bar):
    d_in = X.shape[1]
    rng = np.random.default_rng(d_in)
    f = _features(d_in, rng)
    Xs = X[:, torch.from_numpy(f).to(X.device)].cpu()           # [n, len(f)]: what these entries depend on
    ii, jj = np.meshgrid(np.arange(len(f)), np.arange(len(f)), indexing="ij")
    want = oracle.hessian_entries(Xs, ii.ravel(), jj.ravel()).reshape(len(f), len(f))
    ft = torch.from_numpy(f).to(H.device)
    got = H[ft][:, ft].cpu().numpy().astype(np.float64)
    norm = np.sqrt(np.outer(np.diag(want), np.diag(want)))
    err = float(np.max(np.abs(got - want) / norm))
    fro = float(np.linalg.norm(got - want) / np.linalg.norm(want))
    print(f"{label}: {len(f) ** 2} entries, max error {err:.2e} of sqrt(H_ii H_jj), relative Frobenius error on them {fro:.2e}")
    assert err <= bar and fro <= 1e-3
    assert B.load().cdq_last_device_status() == 0


@pytest.mark.parametrize("n,d_in", [(2048, 4096), (1024, 14336), (512, 18432), (1000, 6152)])
def test_many_tiles_few_rows(n, d_in):
    """Tile counts, tile order (several bands of tile rows) and the single-split path of the large layers, on few
    rows; also: symmetric bit for bit, and two row chunks accumulate to the one-call result."""
    cfg = inputs.CONFIGS["C3"].scaled(d_in=d_in, d_out=8, n=n, seed=500 + d_in % 97)
    X = inputs.make_x(cfg, device="cuda:0")
    H = B.cdq_hessian(X)
    _check(X, H, f"n={n} d_in={d_in}", 1e-5)
    assert torch.equal(H, H.T)
    half = (n // 2) // 64 * 64
    H2 = B.cdq_hessian(X[:half].contiguous())
    H2 = B.cdq_hessian(X[half:].contiguous(), accumulate=True, out=H2)
    assert float((H2 - H).abs().max() / H.diagonal().max()) <= 1e-5


@pytest.mark.parametrize("name", ["C3", "C4"])
def test_full_calibration_set_of_the_benchmark_layers(name):
    cfg = inputs.CONFIGS[name]
    X = inputs.make_x(cfg, device="cuda:0")                     # all n rows (3.8 GB / 9.7 GB of bf16)
    H = B.cdq_hessian(X)
    _check(X, H, f"{name} n={cfg.n} d_in={cfg.d_in}", 1e-4)
    # symmetric bit for bit (checked in row blocks: the transposed copy of a 1.4 GB matrix is not needed whole)
    for r0 in range(0, cfg.d_in, 2048):
        blk = H[r0:r0 + 2048]
        assert torch.equal(blk, H[:, r0:r0 + 2048].T)
    del X, H
    torch.cuda.empty_cache()
