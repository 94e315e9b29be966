"""Multi-GPU plumbing of the benchmark: one process per GPU, no data-path collective.

The path partitions into independent problems (columns, and whole layers), so every rank
quantizes its own layer and the only communication is the barrier around the timed region
and the reduction of the timings (max over ranks) and of the work done (sum over ranks).
The functions take the process group's device so that they run under NCCL on GPUs and under
gloo on CPU (tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the layer a rank works on: distinct layers, reproducible per rank."""
    return base_seed + 1000 * rank


def barrier(world: int, cuda: bool = True) -> None:
    if world > 1:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def aggregate(times_ms, work, world: int, device) -> tuple[list[float], float]:
    """(max over ranks of every entry of times_ms, sum over ranks of work)."""
    if world <= 1:
        return [float(t) for t in times_ms], float(work)
    t = torch.tensor([float(x) for x in times_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([float(work)], dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return t.tolist(), c.item()


def whole_job_throughput(work_all: float, max_ms_total: float, steps: int) -> float:
    """Units per second of the whole job: work of all ranks over the slowest rank's time per step."""
    return work_all / (max_ms_total / steps * 1e-3)
