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


# ---------------------------------------------------------------------------
# One layer over several GPUs (the paper's setting of several accelerators per model): the
# calibration rows are cut into one contiguous shard per rank for the Hessian, which is a sum
# over rows and so needs one all-reduce of d_in^2 fp32 values; the output columns are cut into
# one contiguous slice per rank for everything after it, which needs no exchange (every column
# is an independent problem that shares H).  The only other collective is the sum of the
# per-rank losses.  The reduced H lands in the rank's own memory before any kernel reads it.

def shard_range(total: int, world: int, rank: int, multiple: int = 1) -> tuple[int, int]:
    """[lo, hi) of `total` items for `rank`: contiguous, disjoint, covering, sizes within one
    `multiple` of each other (the last rank takes the ragged end)."""
    assert 0 <= rank < world and total >= 0 and multiple >= 1
    units = (total + multiple - 1) // multiple
    base, extra = divmod(units, world)
    lo_u = rank * base + min(rank, extra)
    hi_u = lo_u + base + (1 if rank < extra else 0)
    return min(lo_u * multiple, total), min(hi_u * multiple, total)


def sharded_layer(lib, X_rows, W_cols, grid, passes: int, world: int, lambda_rel: float = 0.0, ws=None) -> dict:
    """One rank's part of quantizing a layer that is shared out over `world` ranks.

    X_rows: this rank's rows of the calibration inputs [n_r, d_in]; W_cols: its columns of the
    weights [d_in, d_out_r].  `lib` is the binding module (cdq_hessian, cdq_hessian_add_lambda,
    cdq_init_rtn, cdq_cd_solve, cdq_layer_loss).  Returns H (the full, regularised Hessian, the
    same on every rank), this rank's scale/zero/Q, its stats and the loss of the whole layer."""
    kw = {} if ws is None else {"ws": ws}
    H = lib.cdq_hessian(X_rows, **kw)
    if world > 1:
        dist.all_reduce(H, op=dist.ReduceOp.SUM)
    if lambda_rel > 0.0:
        lib.cdq_hessian_add_lambda(H, lambda_rel)
    scale, zero, Q, gamma = lib.cdq_init_rtn(W_cols, grid, H=H if grid.n_clip > 1 else None, **kw)
    stats = lib.cdq_cd_solve(H, W_cols, grid, scale, zero, Q, passes, **kw)
    loss_mine = lib.cdq_layer_loss(H, W_cols, grid, scale, zero, Q, **kw)
    loss = torch.tensor([float(loss_mine)], dtype=torch.float64, device=H.device)
    if world > 1:
        dist.all_reduce(loss, op=dist.ReduceOp.SUM)
    return {"H": H, "scale": scale, "zero": zero, "Q": Q, "gamma": gamma, "stats": stats,
            "loss_mine": float(loss_mine), "loss": float(loss.item())}
