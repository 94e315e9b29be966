"""The benchmark's multi-rank plumbing on CPU: two gloo ranks, no GPU.

The path shards into independent layers (no data-path collective), so what there is to check is
the host logic: distinct per-rank seeds, max-over-ranks timing, summed work, and the whole-job
throughput computed from them."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2406_17542_b200 import inputs, multi


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = inputs.CONFIGS["C0"].scaled(d_in=32, d_out=8, n=64, seed=multi.rank_seed(5, rank))
        X, W = inputs.make_layer(cfg)
        multi.barrier(world, cuda=False)
        # each rank reports its own time and work; rank 1 is the slow one
        times, work = multi.aggregate([10.0 + 5.0 * rank, 20.0 - rank], 100 * (rank + 1), world, "cpu")
        out.put((rank, times, work, float(X.double().sum()), float(W.double().sum())))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_max_time_and_summed_work():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, w0, x0, ww0), (r1, t1, w1, x1, ww1) = res
    assert t0 == t1 == [15.0, 20.0]            # max over ranks, entry by entry
    assert w0 == w1 == 300.0                   # sum over ranks
    assert x0 != x1 and ww0 != ww1             # every rank works on its own layer
    assert multi.whole_job_throughput(w0, t0[0], steps=3) == pytest.approx(300.0 / (15.0 / 3 * 1e-3))


def test_single_rank_needs_no_process_group():
    times, work = multi.aggregate([1.5, 2.5], 7, 1, "cpu")
    assert times == [1.5, 2.5] and work == 7.0
    assert multi.rank_seed(3, 0) == 3 and multi.rank_seed(3, 2) != multi.rank_seed(3, 1)
