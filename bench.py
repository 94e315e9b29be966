#!/usr/bin/env python
"""Benchmark of the CDQuant hot path on B200: one "step" is one pass of the whole path
(Hessian, grid + codes, greedy coordinate descent, layer loss) over one synthetic layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C1] [--impl ours|reference]

Prints ONE JSON line.  `value` is committed coordinate updates per second over the whole
step with inputs resident in HBM; `e2e` is the same with pinned HOST inputs copied in and
the codes, scales and zeros copied back inside the timed region.  `roofline` describes the
dominant kernel (the descent kernel); `cpu_baseline` is the fp64 CPU oracle timed on a
bounded sample of the same workload.  With --impl reference the oracle itself is the timed
program (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2406_17542_b200 import inputs, multi  # noqa: E402

METRIC = "cd_coordinate_updates_per_s"
UNIT = "updates/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the descent kernel, from the ncu
# capture summarised under profiles/ (workload -> bytes); None until a capture exists.
NCU_TRAFFIC_BYTES = {
    # cd_fast_kernel, 4096-column capture (1.784 GB) x 16 254 834 / 4 053 277 committed moves
    "C1": 7.15e9,
    # cd_tma_kernel, 592-column capture (242.5 GB) x 18 354 343 / 5 450 779 committed moves
    "C3": 8.17e11,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx = float(f[2])
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        # median over the upper half of the samples = under load (idle samples sit at the low end)
        load = sm[len(sm) // 2:] if sm else []
        med = load[len(load) // 2] if load else None
        return {"sm_mhz": med, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm)}


def kernel_launches(cfg) -> int:
    """Kernels of the library launched by one step (counted from the launch sequences in csrc/)."""
    tc_h = cfg.x_dtype == "bf16" and cfg.n >= 256 and cfg.d_in >= 256          # tcgen05 Hessian: order, MMA, reduce
    tc_g = cfg.d_in >= 256 and cfg.d_out >= 128                                  # int8 tensor-core H E
    hessian = 3 if tc_h else 1
    prep_h = 2                                                                   # row exponents, slices of H
    he = 5 if tc_g else 2                # column max, exponents, slices of E^T, GEMM, sum of the column dots | GEMM, partial sums
    init = 5                                                                     # min/max x2, gamma fill or argmin, scale/zero, codes
    if cfg.n_clip > 1:
        init += (prep_h if tc_g else 0) + cfg.n_clip * (1 + he)                  # per gamma: residual + H E
    cd = 1 + (prep_h if tc_g else 0) + he + 1 + 1 + 1 + 1 + 1                    # residual, H E, sum, transpose, diag, descent, transpose
    loss = 1 + (prep_h if tc_g else 0) + he + 1                                  # residual, H E, sum
    return hessian + init + cd + loss


def algorithmic_bytes_cd(cfg, committed: int) -> float:
    """Descent kernel: one fp32 row of H per committed move, plus per-column state in and out
    (fp64 gradient in, codes in and out, scales)."""
    ng = cfg.d_in // cfg.group_size if cfg.group_size else 1
    per_col = 8 * cfg.d_in + 2 * cfg.d_in + 4 * ng
    return committed * 4.0 * cfg.d_in + cfg.d_out * float(per_col)


def run_oracle_sample(cfg, X, W, n_rows: int, n_cols: int) -> dict:
    """The CPU oracle, as it stands, on a bounded sample: the first n_rows calibration rows and
    n_cols evenly spaced columns; stage times are extrapolated to the full layer."""
    import oracle
    Xs = X[:n_rows].cpu()
    step = max(cfg.d_out // n_cols, 1)
    cols = torch.arange(0, cfg.d_out, step)[:n_cols]
    Ws = W[:, cols.to(W.device)].cpu()
    t0 = time.perf_counter()
    _, H32 = oracle.hessian(Xs)
    t_h = time.perf_counter() - t0
    t0 = time.perf_counter()
    init = oracle.init_rtn(Ws, cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi,
                           H=H32 if cfg.n_clip > 1 else None)
    res = oracle.cd_solve(H32, Ws, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in,
                          cfg.group_size)
    oracle.layer_loss(H32, Ws, init["scale"], init["zero"], res["Q"], cfg.group_size)
    t_c = time.perf_counter() - t0
    t_full = t_h * (cfg.n / n_rows) + t_c * (cfg.d_out / len(cols))
    committed_full = res["committed"] * (cfg.d_out / len(cols))
    return {"value": committed_full / t_full, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n_rows} of {cfg.n} rows for H ({t_h:.2f} s), {len(cols)} of {cfg.d_out} columns for "
                      f"grid+CD+loss ({t_c:.2f} s); extrapolated to the full layer ({t_full:.1f} s)",
            "seconds_per_layer_extrapolated": t_full, "measured_s": t_h + t_c}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="C1", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--budget-div", type=int, default=0,
                    help="descent budget T = d_in / DIV steps per column (the paper's fewer-iterations study) "
                         "instead of the config's passes * d_in")
    ap.add_argument("--block", type=int, default=1, choices=[1, 2],
                    help="1: greedy descent (the headline path); 2: the greedy descent followed by BCD with random pairs "
                         "(Algorithm 2 / 5; T = d_in steps per column, or d_in / --budget-div); the roofline object then "
                         "describes the BCD kernel and no CPU baseline is timed")
    ap.add_argument("--init", default="rtn", choices=["rtn", "owc_cd"],
                    help="grid stage: cdq_init_rtn (MinMax / OWC as the config says) or cdq_init_owc_cd (Algorithm 3; "
                         "configs with a clipping grid)")
    ap.add_argument("--shard", action="store_true",
                    help="share ONE layer out over the ranks (strong scaling): rows of X per rank for the Hessian with one "
                         "all-reduce, columns of W per rank after it; the default gives every rank its own layer (weak)")
    ap.add_argument("--d-out", type=int, default=0, help="profiling case: keep only this many output columns")
    ap.add_argument("--n", type=int, default=0, help="profiling case: keep only this many calibration rows")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = inputs.CONFIGS[args.config]
    if args.d_out or args.n:
        cfg = cfg.scaled(d_out=args.d_out or cfg.d_out, n=args.n or cfg.n)
    if args.init == "owc_cd" and cfg.n_clip < 2:
        ap.error("--init owc_cd needs a config with a clipping grid (C2, C4)")
    workload = (f"{cfg.name}: d_in={cfg.d_in} d_out={cfg.d_out} n={cfg.n} X={cfg.x_dtype} W={cfg.w_dtype} "
                f"bits={cfg.bits} group={cfg.group_size or 'per-channel'} n_clip={cfg.n_clip} passes={cfg.passes}"
                + (" init=OWC-CD" if args.init == "owc_cd" else "")
                + (f" budget=d_in/{args.budget_div}" if args.budget_div > 0 else "")
                + (" descent=CD then BCD(k=2)" if args.block == 2 else ""))

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, cfg, workload)
        return

    from paper_2406_17542_b200 import binding as B
    B.load()  # fails loudly when the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # every rank quantizes its own layer (same shape, its own seed): columns and layers are
    # independent problems, so there is no data-path collective
    my_cfg = cfg if args.shard else cfg.scaled(seed=multi.rank_seed(cfg.seed, rank))
    X, W = inputs.make_layer(my_cfg, device=dev)
    if args.shard:   # the same layer everywhere; this rank keeps its rows of X and its columns of W
        r0, r1 = multi.shard_range(cfg.n, world, rank, multiple=64)
        c0, c1 = multi.shard_range(cfg.d_out, world, rank)
        X, W = X[r0:r1].contiguous(), W[:, c0:c1].contiguous()
    Xh, Wh = X.cpu().pin_memory(), W.cpu().pin_memory()
    grid = B.Grid(cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi)
    ws = B.Workspace()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def barrier():
        multi.barrier(world)

    pinned_out: list = []

    def one_step(host: bool, times: dict | None = None):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        ev[0].record()
        Xd = Xh.to(dev, non_blocking=True) if host else X
        Wd = Wh.to(dev, non_blocking=True) if host else W
        ev[1].record()
        H = B.cdq_hessian(Xd, ws=ws)
        if args.shard and world > 1:   # the one exchange of the sharded layer: sum of the row shards' Hessians
            dist.all_reduce(H, op=dist.ReduceOp.SUM)
        ev[2].record()
        if args.init == "owc_cd":
            scale, zero, Q, _, _ = B.cdq_init_owc_cd(Wd, grid, H, ws=ws)
        else:
            scale, zero, Q, _ = B.cdq_init_rtn(Wd, grid, H=H if cfg.n_clip > 1 else None, ws=ws)
        ev[3].record()
        budget = cfg.d_in // args.budget_div if args.budget_div > 0 else None
        stats = B.cdq_cd_solve(H, Wd, grid, scale, zero, Q, cfg.passes, ws=ws,
                               steps_per_col=budget if args.block == 1 else None)
        if args.block == 2:  # the paper starts BCD from the greedy solution
            cd_stats = stats
            stats = B.cdq_bcd_solve(H, Wd, grid, scale, zero, Q, 2, budget or cfg.d_in, seed=cfg.seed, ws=ws)
            stats["cd_kernel_ms_before_bcd"] = cd_stats["kernel_ms"]
            stats["loss_after_cd"] = cd_stats["loss_after"]
        ev[4].record()
        loss = B.cdq_layer_loss(H, Wd, grid, scale, zero, Q, ws=ws)
        if host:   # results back into pinned host buffers (allocated once, reused every step)
            srcs = (Q, scale, zero)
            if not pinned_out:
                pinned_out.extend(torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in srcs)
            for dst, src in zip(pinned_out, srcs):
                dst.copy_(src, non_blocking=True)
            d2h = sum(t.numel() * t.element_size() for t in srcs) + 8
        else:
            d2h = 0
        ev[5].record()
        torch.cuda.synchronize()
        if times is not None:
            for name, a, b in (("copy_in", 0, 1), ("hessian", 1, 2), ("init_rtn", 2, 3), ("cd_solve", 3, 4),
                               ("loss_and_copy_out", 4, 5), ("total", 0, 5)):
                times.setdefault(name, []).append(ev[a].elapsed_time(ev[b]))
            times.setdefault("cd_kernel", []).append(stats["kernel_ms"])
        return stats, loss, d2h

    def timed(host: bool):
        for _ in range(max(args.warmup, 0)):
            one_step(host)
        times: dict = {}
        stats = loss = None
        d2h = 0
        barrier()
        for _ in range(args.steps):
            flush.fill_(1)           # evict L2 between timed iterations (not timed)
            torch.cuda.synchronize()
            stats, loss, d2h = one_step(host, times)
        barrier()
        return times, stats, loss, d2h

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    times, stats, loss, _ = timed(host=False)
    clocks = sampler.stop() if sampler else None
    times_e2e, stats_e2e, _, d2h = timed(host=True)

    total_ms = sum(times["total"])
    total_ms_e2e = sum(times_e2e["total"])
    committed = stats["committed"]
    (total_ms, total_ms_e2e), committed_all = multi.aggregate([total_ms, total_ms_e2e], committed, world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    acc = cfg.scaled(d_out=W.shape[1], n=X.shape[0])   # what this rank worked on (the whole layer unless --shard)
    ms_per_step = total_ms / args.steps
    value = multi.whole_job_throughput(committed_all, total_ms, args.steps)
    mean = lambda v: sum(v) / len(v)
    cd_ms = mean(times["cd_kernel"])
    alg_bytes = algorithmic_bytes_cd(acc, committed)
    if args.block == 2:  # two rows per move at most, and one H_im per pair and step
        alg_bytes += committed * 4.0 * cfg.d_in + stats["steps"] * 2.0 * cfg.d_in
    achieved = alg_bytes / (cd_ms * 1e-3) / 1e9
    h_in_l2 = 4.0 * cfg.d_in * cfg.d_in < 100e6
    hess_ms = mean(times["hessian"])
    hess_flops = 2.0 * acc.n * cfg.d_in * cfg.d_in
    # flops the tensor cores actually execute: 128 x 256 tiles that touch the lower triangle
    # (tile (tm, tn) with tn <= tm // 2), over the rows padded to the 64-row K block
    tiles_m = (cfg.d_in + 127) // 128
    n_tiles = sum(tm // 2 + 1 for tm in range(tiles_m))
    hess_exec = 2.0 * 128 * 256 * n_tiles * ((acc.n + 63) // 64 * 64) if cfg.x_dtype == "bf16" and cfg.d_in >= 256 else hess_flops
    h2d = Xh.numel() * Xh.element_size() + Wh.numel() * Wh.element_size()
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if args.shard else "weak", "vs_baseline": None,
        "dtype": "f32 scores / f64 gradient / bf16 Hessian inputs", "data": "synthetic",
        "config": {"workload": workload, "l2": "256 MiB flush between timed iterations; X also exceeds L2",
                   "per_rank": ("one layer shared out: row shards of X + one all-reduce of H, column slices of W after it"
                                if args.shard else "one independent layer per GPU, no collective")},
        "sec_per_layer": ms_per_step * 1e-3,
        "cd": {"committed_updates": committed, "step_budget": stats["steps"],
               "columns_converged": stats["columns_converged"], "kernel_ms": cd_ms,
               "committed_updates_per_s_kernel": committed / (cd_ms * 1e-3),
               "budget_steps_per_s_kernel": stats["steps"] / (cd_ms * 1e-3),
               "loss_before": stats["loss_before"], "loss_after": stats["loss_after"], "loss": loss,
               **({"cd_kernel_ms_before_bcd": stats["cd_kernel_ms_before_bcd"], "loss_after_cd": stats["loss_after_cd"]}
                  if args.block == 2 else {})},
        "stages_ms": {k: mean(v) for k, v in times.items()},
        "hessian": {"ms": hess_ms, "dense_equivalent_tflops": hess_flops / (hess_ms * 1e-3) / 1e12,
                    "executed_tflops": hess_exec / (hess_ms * 1e-3) / 1e12,
                    "executed_frac_of_bf16_sustained_peak": hess_exec / (hess_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                    "executed_frac_of_bf16_burst_peak": hess_exec / (hess_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "note": "symmetric rank-k update: only lower-triangle tiles are computed; the fraction counts executed flops only"},
        "roofline": {"kernel": "bcd2_kernel" if args.block == 2 else ("cd_tma_kernel" if cfg.d_in > 2048 and cfg.d_in % 4 == 0
                                                                  else "cd_fast_kernel"), "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "traffic": NCU_TRAFFIC_BYTES.get(cfg.name) if args.block == 1 else None, "algorithmic_bytes": alg_bytes,
                     "note": ("H fits in L2 for this workload: rows are L2-served, the figure is effective GB/s"
                              if h_in_l2 else "H exceeds L2: rows stream from HBM")},
        "e2e": {"value": committed_all / (total_ms_e2e / args.steps * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": total_ms_e2e / args.steps},
        "gpu_launches": kernel_launches(acc) * args.steps,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline and args.block == 1:
        # about 5-10 s of Hessian and 5-10 s of descent on 8 host cores
        n_rows = min(cfg.n, max(1024, int(4.0e10 / (cfg.d_in * cfg.d_in))))
        n_cols = min(cfg.d_out, max(8, int(3.0e10 / (0.8 * cfg.d_in * cfg.d_in * (2 ** cfg.bits)))))
        out["cpu_baseline"] = run_oracle_sample(cfg, X, W, n_rows, n_cols)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_reference(args, cfg, workload):
    """The oracle as the timed program: each step is one bounded sample of the workload."""
    import oracle
    X, W = inputs.make_layer(cfg.scaled(n=min(cfg.n, 4096)), device="cpu")
    n_rows = min(cfg.n, 2048)
    n_cols = min(cfg.d_out, 32)
    for _ in range(max(args.warmup, 0)):
        run_oracle_sample(cfg, X, W, n_rows, n_cols)
    vals, secs = [], []
    r = None
    for _ in range(args.steps):
        r = run_oracle_sample(cfg, X, W, n_rows, n_cols)
        vals.append(r["value"]); secs.append(r["measured_s"])
    value = sum(vals) / len(vals)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": r["cores"], "kind": "oracle", "sample": r["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    main()
