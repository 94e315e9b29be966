"""cdq_cd_solve_rows16: the greedy descent reading its rows from a bf16 copy of H (half the bytes per move).

Two gates.  (i) The kernel: the call is defined as the descent on H' (off-diagonal entries of H rounded to bf16,
diagonal exact), so the oracle, given H', must produce the same codes -- the usual production-mode bars (every
column equal or an audited fp32 near-tie fork, column losses on H' within 1e-4).  (ii) What it costs: the loss on
the true H of the bf16-row result against that of the fp32-row result, printed and bounded."""
import numpy as np
import pytest
import torch

from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs
from tests.util import compare_with_oracle, grid_of

pytestmark = pytest.mark.gpu


def _rounded(Hd):
    Hr = Hd.to(torch.bfloat16).to(torch.float32)
    Hr.diagonal().copy_(Hd.diagonal())
    return Hr.contiguous()


def _h_from_rows(cfg, rows, ridge=1e-3):
    X = inputs.make_x(cfg.scaled(n=rows), device="cuda:0").double()
    H = X.T @ X
    H += ridge * H.diagonal().mean() * torch.eye(cfg.d_in, dtype=torch.float64, device=H.device)
    return H.float().contiguous()


@pytest.mark.parametrize("name,d_in,d_out,g,bits,rows,n_sample", [
    ("C3", 4608, 64, 0, 4, 4096, 64),          # two 256-thread teams per SM
    ("C3", 6144, 148, 0, 3, 4096, 32),
    ("C3", 11008, 148, 0, 4, 4096, 16),        # ragged: the last chunk slots reach past the row
    ("C3", 14336, 296, 0, 4, 8192, 24),        # the C3 team (256 threads x 14 chunks)
    ("C4", 18432, 148, 128, 3, 4096, 12),      # the C4 team (384 threads x 12 chunks), groups of 128
])
def test_bf16_rows_against_the_oracle_on_the_rounded_matrix(name, d_in, d_out, g, bits, rows, n_sample):
    cfg = inputs.CONFIGS[name].scaled(d_in=d_in, d_out=d_out, group_size=g, bits=bits, n_clip=1, clip_lo=1.0, clip_hi=1.0,
                                      passes=1, seed=800 + d_in % 89)
    dev = "cuda:0"
    Hd = _h_from_rows(cfg, rows)
    Wd = inputs.make_w(cfg, device=dev)
    gd = grid_of(cfg)
    scale, zero, Q0, gamma = B.cdq_init_rtn(Wd, gd)
    Q = Q0.clone()
    st = B.cdq_cd_solve(Hd, Wd, gd, scale, zero, Q, cfg.passes, rows16=True)
    assert B.load().cdq_last_device_status() == 0
    Hr = _rounded(Hd)
    loss_r, per_r = B.cdq_layer_loss(Hr, Wd, gd, scale, zero, Q, per_col=True)        # on H': what the call minimises
    np.testing.assert_allclose(st["loss_after"], loss_r, rtol=1e-5)
    cols = np.sort(np.random.default_rng(d_in).choice(d_out, n_sample, replace=False))
    compare_with_oracle(cfg, Hr.cpu().numpy(), Hd, Wd, cols, gd, scale, zero, Q0, Q, gamma, per_r, cfg.passes * d_in,
                        label=f"rows16 {d_in}x{d_out}", rows16=True)
    # (ii) the price on the true objective
    Q32 = Q0.clone()
    B.cdq_cd_solve(Hd, Wd, gd, scale, zero, Q32, cfg.passes)
    l16 = B.cdq_layer_loss(Hd, Wd, gd, scale, zero, Q)
    l32 = B.cdq_layer_loss(Hd, Wd, gd, scale, zero, Q32)
    l0 = B.cdq_layer_loss(Hd, Wd, gd, scale, zero, Q0)
    print(f"rows16 {d_in}x{d_out}: loss on H after the descent: fp32 rows {l32:.6g}, bf16 rows {l16:.6g} "
          f"(ratio {l16 / l32:.5f}); round-to-nearest start {l0:.6g}")
    assert l16 <= 1.02 * l32 and l16 < l0


def test_shapes_without_a_bf16_row_kernel_are_refused():
    for d_in, g in ((1024, 0), (4100, 0), (4608, 6)):
        cfg = inputs.CONFIGS["C0"].scaled(d_in=d_in, d_out=8, n=64, group_size=g, bits=3)
        dev = "cuda:0"
        Hd = torch.eye(d_in, device=dev)
        Wd = inputs.make_w(cfg, device=dev)
        gd = grid_of(cfg)
        scale, zero, Q, _ = B.cdq_init_rtn(Wd, gd)
        with pytest.raises(B.CdqError) as err:
            B.cdq_cd_solve(Hd, Wd, gd, scale, zero, Q, 1, rows16=True)
        assert err.value.status == 3
