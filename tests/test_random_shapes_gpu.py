"""Seeded random small layers (odd sizes, 1..5 bits, group sizes from 1 up, fewer rows than features, clipping
grids) through every entry point in the fp64 verification mode: H, grid and codes, greedy descent, pairs and
OWC-CD have to equal the oracle bit for bit on each of them."""
import random

import numpy as np
import pytest
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs

pytestmark = pytest.mark.gpu


def _case(rng, it):
    d_in = rng.choice([1, 2, 3, 8, 12, 30, 33, 64, 96, 128, 200, 256, 320])
    d_out = rng.choice([1, 2, 7, 33, 64])
    bits = rng.choice([1, 2, 3, 4, 5])
    divs = [g for g in (1, 2, 3, 4, 5, 8, 10, 16, 32, 64) if d_in % g == 0 and g < d_in]
    g = rng.choice([0] + divs) if divs else 0
    n = rng.choice([3, max(4, d_in // 2), d_in + 7])
    n_clip = rng.choice([1, 4])
    return inputs.CONFIGS["C0"].scaled(d_in=d_in, d_out=d_out, n=n, bits=bits, group_size=g, passes=2, seed=5000 + it,
                                       n_clip=n_clip, clip_lo=0.5, clip_hi=1.0)


@pytest.mark.parametrize("block", range(4))
def test_random_small_layers_verify_mode(block):
    rng = random.Random(100 + block)
    for it in range(12):
        cfg = _case(rng, 100 * block + it)
        tag = f"{cfg.d_in}x{cfg.d_out} n={cfg.n} bits={cfg.bits} g={cfg.group_size} clip={cfg.n_clip}"
        X, W = inputs.make_layer(cfg)
        _, H32 = oracle.hessian(X, 0.0)
        assert np.array_equal(B.cdq_hessian(X.cuda(), mode="verify").cpu().numpy(), H32), tag
        Hd, Wd = torch.from_numpy(H32).cuda(), W.cuda()
        grid = B.Grid(cfg.bits, cfg.group_size, cfg.n_clip, 0.5, 1.0)
        use_h = cfg.n_clip > 1
        init = oracle.init_rtn(W, cfg.bits, cfg.group_size, cfg.n_clip, 0.5, 1.0, H=H32 if use_h else None)
        scale, zero, Q, _ = B.cdq_init_rtn(Wd, grid, H=Hd if use_h else None, mode="verify")
        assert np.array_equal(Q.cpu().numpy(), init["Q"]) and np.array_equal(scale.cpu().numpy(), init["scale"]), tag
        ref = oracle.cd_solve(H32, W, cfg.bits, init["scale"], init["zero"], init["Q"], 2 * cfg.d_in, cfg.group_size)
        B.cdq_cd_solve(Hd, Wd, grid, scale, zero, Q, 2, mode="verify")
        assert np.array_equal(Q.cpu().numpy(), ref["Q"]), tag
        if cfg.d_in % 2 == 0:
            T = min(40, 2 * cfg.d_in)
            refb = oracle.bcd_solve(H32, W, cfg.bits, init["scale"], init["zero"], ref["Q"], 2, T, seed=it,
                                    group_size=cfg.group_size)
            B.cdq_bcd_solve(Hd, Wd, grid, scale, zero, Q, 2, T, seed=it, mode="verify")
            assert np.array_equal(Q.cpu().numpy(), refb["Q"]), tag
        if use_h and cfg.group_size:
            ro = oracle.owc_cd(H32, W, cfg.bits, cfg.group_size, cfg.n_clip, 0.5, 1.0, steps=cfg.d_in // cfg.group_size)
            s2, _, Q2, _, _ = B.cdq_init_owc_cd(Wd, grid, Hd, mode="verify")
            assert np.array_equal(Q2.cpu().numpy(), ro["Q"]) and np.array_equal(s2.cpu().numpy(), ro["scale"]), tag
    assert B.load().cdq_last_device_status() == 0
