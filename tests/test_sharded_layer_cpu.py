"""One layer shared out over two ranks, on CPU with gloo: rows of X per rank for the Hessian
(one all-reduce), columns of W per rank for everything after it (no exchange).

The CUDA library cannot run here, so the ranks drive a stand-in with the binding's function
names whose bodies are the CPU oracle; what is under test is the sharding itself: the ranges,
the all-reduce, the regulariser applied once to the sum, and that the two ranks' column slices
put together are the unsharded result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2406_17542_b200 import inputs, multi


class Grid:
    def __init__(self, bits, group_size=0, n_clip=1, clip_lo=1.0, clip_hi=1.0):
        self.bits, self.group_size, self.n_clip, self.clip_lo, self.clip_hi = bits, group_size, n_clip, clip_lo, clip_hi


class OracleLib:
    """The binding's names on CPU tensors (part Hessians are plain fp32 sums of outer products)."""

    @staticmethod
    def cdq_hessian(X):
        Xd = X.double()
        return (Xd.T @ Xd).float().contiguous()

    @staticmethod
    def cdq_hessian_add_lambda(H, lambda_rel):
        H.diagonal().add_(float(lambda_rel) * float(H.diagonal().double().mean()))
        return H

    @staticmethod
    def cdq_init_rtn(W, grid, H=None):
        r = oracle.init_rtn(W, grid.bits, grid.group_size, grid.n_clip, grid.clip_lo, grid.clip_hi,
                            H=None if H is None else H.numpy())
        return torch.from_numpy(r["scale"]), torch.from_numpy(r["zero"]), torch.from_numpy(r["Q"]), None

    @staticmethod
    def cdq_cd_solve(H, W, grid, scale, zero, Q, passes):
        r = oracle.cd_solve(H.numpy(), W, grid.bits, scale.numpy(), zero.numpy(), Q.numpy(), passes * W.shape[0],
                            grid.group_size)
        Q.copy_(torch.from_numpy(r["Q"]))
        return {"committed": int(r["committed"])}

    @staticmethod
    def cdq_layer_loss(H, W, grid, scale, zero, Q):
        total, _ = oracle.layer_loss(H.numpy(), W, scale.numpy(), zero.numpy(), Q.numpy(), grid.group_size)
        return float(total)


CFG = dict(d_in=48, d_out=22, n=203, bits=3, group_size=16, passes=1, seed=31)
LAMBDA = 0.01


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = inputs.CONFIGS["C0"].scaled(**CFG)
        X, W = inputs.make_layer(cfg)                       # the same layer on every rank
        r0, r1 = multi.shard_range(cfg.n, world, rank, multiple=64)
        c0, c1 = multi.shard_range(cfg.d_out, world, rank)
        res = multi.sharded_layer(OracleLib, X[r0:r1], W[:, c0:c1].contiguous(), Grid(cfg.bits, cfg.group_size),
                                  cfg.passes, world, lambda_rel=LAMBDA)
        out.put((rank, (r0, r1), (c0, c1), res["H"].numpy(), res["Q"].numpy(), res["loss"], res["loss_mine"],
                 res["stats"]["committed"]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_share_one_layer():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, rows0, cols0, H0, Q0, loss0, mine0, m0), (_, rows1, cols1, H1, Q1, loss1, mine1, m1) = res
    cfg = inputs.CONFIGS["C0"].scaled(**CFG)
    assert rows0 == (0, 128) and rows1 == (128, cfg.n)        # shards in multiples of 64 rows, ragged end last
    assert cols0 == (0, 11) and cols1 == (11, 22)
    assert np.array_equal(H0, H1)                              # every rank holds the same reduced H
    assert loss0 == loss1 == pytest.approx(mine0 + mine1, rel=1e-12)

    # the unsharded layer with the same (reduced, regularised) H
    X, W = inputs.make_layer(cfg)
    Hfull = OracleLib.cdq_hessian_add_lambda(OracleLib.cdq_hessian(X), LAMBDA).numpy()
    np.testing.assert_allclose(H0, Hfull, rtol=2e-6, atol=1e-6 * np.abs(Hfull).max())
    assert H0[0, 0] > (X[:, 0].double() ** 2).sum().item()    # the regulariser went in, once
    init = oracle.init_rtn(W, cfg.bits, cfg.group_size, 1, 1.0, 1.0)
    cd = oracle.cd_solve(H0, W, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in, cfg.group_size)
    assert np.array_equal(np.concatenate([Q0, Q1], axis=1), cd["Q"])
    assert m0 + m1 == int(cd["committed"])
    total, _ = oracle.layer_loss(H0, W, init["scale"], init["zero"], cd["Q"], cfg.group_size)
    assert loss0 == pytest.approx(total, rel=1e-12)


def test_shard_ranges_cover_without_overlap():
    for total, world, mult in ((0, 3, 1), (5, 8, 1), (203, 2, 64), (65536, 8, 64), (1000, 3, 64), (7, 7, 1)):
        spans = [multi.shard_range(total, world, r, mult) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == total
        for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
            assert a1 == b0 and a0 <= a1
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= mult + (total % mult if mult > 1 else 0)
