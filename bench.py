#!/usr/bin/env python
"""Benchmark of the CDQuant hot path on B200: one "step" is one pass of the whole path
(Hessian, grid + codes, greedy coordinate descent, layer loss) over one synthetic layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C3] [--impl ours|reference]

Prints ONE JSON line.  `value` is committed coordinate updates per second over the whole
step with inputs resident in HBM; `e2e` is the same with pinned HOST inputs copied in and
the codes, scales and zeros copied back inside the timed region.  `roofline` describes the
dominant kernel (the descent kernel) and says what serves the rows of H: "hbm" when H is larger
than L2 (then `frac` is a fraction of the measured HBM copy bandwidth), "l2" when H sits in L2
(then the figure is an effective rate and no fraction of the HBM peak is claimed).
`parity` compares, in the same run and with the run's own H, the codes and column losses of a
seeded sample of columns with the fp64 CPU oracle; `cpu_baseline` is that oracle timed on a
bounded sample of the same workload.  `other_configs` holds the same record (without the
end-to-end leg) for the other benchmark layers at one warm-up and one timed step each.
With --impl reference the oracle itself is the timed program (rank 0 only).
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2406_17542_b200 import inputs, multi  # noqa: E402

METRIC = "cd_coordinate_updates_per_s"
UNIT = "updates/s"
L2_BYTES = 126e6

# DRAM bytes per committed move of the descent kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture divided by the moves of that capture), keyed by (kernel, d_in); a kernel and shape without a
# capture of the kernel as it stands reports traffic null.  Each entry names the summary it comes from.
NCU_TRAFFIC_PER_MOVE: dict = {
    ("cd_tma_kernel", 14336): (44533.0, "profiles/cd_tma_kernel_C3_592cols.md"),
}


def descent_kernel_name(cfg, block: int) -> str:
    if block == 2:
        return "bcd2_kernel"
    return "cd_tma_kernel" if cfg.d_in > 1536 and cfg.d_in % 4 == 0 else "cd_fast_kernel"


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


def algorithmic_bytes_cd(cfg, committed: int, row_bytes: float = 4.0) -> float:
    """Descent kernel: one row of H per committed move (fp32, or bf16 with --rows16), plus per-column state in
    and out (fp64 gradient in, codes in and out, scales)."""
    ng = cfg.d_in // cfg.group_size if cfg.group_size else 1
    per_col = 8 * cfg.d_in + 2 * cfg.d_in + 4 * ng
    return committed * row_bytes * cfg.d_in + cfg.d_out * float(per_col)


def run_oracle_sample(cfg, X, W, n_rows: int, n_cols: int) -> dict:
    """The CPU oracle, as it stands, on a bounded sample: the first n_rows calibration rows and
    n_cols evenly spaced columns; stage times are extrapolated to the full layer."""
    import oracle
    n_rows, n_cols = min(n_rows, X.shape[0]), min(n_cols, W.shape[1])   # (X, W may be a slice of the layer already)
    Xs = X[:n_rows].cpu()
    step = max(W.shape[1] // n_cols, 1)
    cols = torch.arange(0, W.shape[1], step)[:n_cols]
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


def baseline_sample_size(cfg) -> tuple:
    """Rows and columns for about 5-10 s of Hessian and 5-10 s of descent on ~8-16 host cores."""
    n_rows = min(cfg.n, max(1024, int(4.0e10 / (cfg.d_in * cfg.d_in))))
    n_cols = min(cfg.d_out, max(8, int(3.0e10 / (0.8 * cfg.d_in * cfg.d_in * (2 ** cfg.bits)))))
    return n_rows, n_cols


def parity_in_run(B, cfg, grid, H, Wd, scale, zero, Q0, Q, gamma, per_col, n_cols: int) -> dict:
    """Codes and column losses of n_cols seeded columns of this run against the oracle with this run's own H.
    A column that differs is audited (oracle/audit.py): it must have left the oracle's trajectory at a step
    the oracle scores as a near-tie below fp32 resolution; with a clipping search, a column whose clipping
    strength differs must be a near-tie of the oracle's own loss table (it is then left out of the code
    comparison: other grid, other codes)."""
    import oracle
    from oracle import audit
    dev = Wd.device
    rng = np.random.default_rng(cfg.seed + 1000)
    cols = np.sort(rng.choice(cfg.d_out, min(n_cols, cfg.d_out), replace=False))
    ct = torch.from_numpy(cols).to(dev)
    t0 = time.perf_counter()
    H32 = H.cpu().numpy()
    Wc = Wd[:, ct].cpu()
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi,
                           H=H32 if cfg.n_clip > 1 else None, want_loss_table=cfg.n_clip > 1)
    keep = np.arange(len(cols))
    gamma_wide = 0
    if cfg.n_clip > 1:
        gg = oracle.gamma_grid(cfg.n_clip, cfg.clip_lo, cfg.clip_hi).astype(np.float32)
        got_gamma = gamma.cpu().numpy()[cols]
        same = got_gamma == gg[init["gamma_idx"]]
        for j in np.nonzero(~same)[0]:
            t = init["loss_table"][:, j]
            k_lib = int(np.argmin(np.abs(gg - got_gamma[j])))
            if abs(t[k_lib] - t[init["gamma_idx"][j]]) > 1e-7 * t[init["gamma_idx"][j]]:
                gamma_wide += 1
        keep = np.nonzero(same)[0]
    budget = cfg.passes * cfg.d_in
    kt = ct[torch.from_numpy(keep).to(dev)]
    Wk = Wc[:, torch.from_numpy(keep)]
    sc, ze, q0 = init["scale"][:, keep], init["zero"][:, keep], init["Q"][:, keep]
    start_equal = bool(np.array_equal(Q0[:, kt].cpu().numpy(), q0) and np.array_equal(scale[:, kt].cpu().numpy(), sc))
    ref = oracle.cd_solve(H32, Wk, cfg.bits, sc, ze, q0, budget, cfg.group_size)
    _, per_ref = oracle.layer_loss(H32, Wk, sc, ze, ref["Q"], cfg.group_size)
    got = Q[:, kt].cpu().numpy()
    Wk_d, sc_d, ze_d, q0_d = Wd[:, kt].contiguous(), scale[:, kt].contiguous(), zero[:, kt].contiguous(), Q0[:, kt].contiguous()
    cache: dict = {}

    def lib_after(j, t):
        if t not in cache:
            Qt = q0_d.clone()
            if t > 0:
                B.cdq_cd_solve(H, Wk_d, grid, sc_d, ze_d, Qt, 0, steps_per_col=int(t))
            cache[t] = Qt.cpu().numpy()
        return cache[t][:, j]

    reports = audit.audit_cd_columns(oracle, H32, Wk, cfg.bits, sc, ze, q0, ref["Q"], got, budget, cfg.group_size, lib_after)
    replay_ok = all(np.array_equal(lib_after(r["col"], budget), got[:, r["col"]]) for r in reports)
    forked = np.array([r["col"] for r in reports], dtype=np.int64)
    rest = np.setdiff1d(np.arange(len(keep)), forked)
    per_got = per_col.cpu().numpy()[cols][keep]
    return {"cols": int(len(cols)), "cols_compared": int(len(keep)),
            "start_codes_and_scales_equal": start_equal,
            "code_agreement": float((got == ref["Q"]).mean()),
            "code_agreement_without_audited_forks": float((got[:, rest] == ref["Q"][:, rest]).mean()) if len(rest) else 1.0,
            "loss_rel": float(abs(per_got.sum() - per_ref.sum()) / per_ref.sum()),
            "forks_audited": int(sum(r["ok"] for r in reports)), "forks_unexplained": int(sum(not r["ok"] for r in reports)),
            "largest_audited_gap": float(max([r["gap"] for r in reports if r["ok"]], default=0.0)),
            "replay_reproduces_run": bool(replay_ok),
            "clip_strength_differs": int(len(cols) - len(keep)), "clip_strength_differs_at_wide_gap": int(gamma_wide),
            "oracle_s": time.perf_counter() - t0}


def run_config(B, cfg, args, steps: int, warmup: int, dev, world: int, rank: int, e2e: bool, parity_cols: int,
               sample_clocks: bool, local_rank: int):
    """Times `steps` steps of one layer after `warmup` untimed ones.  Returns the record of this configuration
    (rank 0) and what the caller needs for the whole-job line."""
    import torch.distributed as dist
    lib = B.load()
    my_cfg = cfg if args.shard else cfg.scaled(seed=multi.rank_seed(cfg.seed, rank))
    X, W = inputs.make_layer(my_cfg, device=dev)
    if args.shard:   # the same layer everywhere; this rank keeps its rows of X and its columns of W
        r0, r1 = multi.shard_range(cfg.n, world, rank, multiple=64)
        c0, c1 = multi.shard_range(cfg.d_out, world, rank)
        X, W = X[r0:r1].contiguous(), W[:, c0:c1].contiguous()
    Xh = Wh = None
    if e2e:
        Xh, Wh = X.cpu().pin_memory(), W.cpu().pin_memory()
    grid = B.Grid(cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi)
    ws = B.Workspace()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    pinned_out: list = []
    keep: dict = {}

    def one_step(host: bool, times: dict | None = None, last: bool = False):
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
            scale, zero, Q, gamma, _ = B.cdq_init_owc_cd(Wd, grid, H, ws=ws)
        else:
            scale, zero, Q, gamma = B.cdq_init_rtn(Wd, grid, H=H if cfg.n_clip > 1 else None, ws=ws)
        ev[3].record()
        # the last timed step keeps what the in-run parity check needs (earlier steps must not: a held H would make
        # the next step allocate a fresh one inside the timed region)
        Q0 = Q.clone() if (last and parity_cols > 0 and not host) else None   # (a copy, not a kernel of the library)
        budget = cfg.d_in // args.budget_div if args.budget_div > 0 else None
        want_cols = Q0 is not None
        per = None
        if args.block == 1 and not args.rows16:
            # the descent returns the loss of its result (half the dot product of residual and final gradient)
            res = B.cdq_cd_solve_with_loss(H, Wd, grid, scale, zero, Q, budget or cfg.passes * cfg.d_in, ws=ws,
                                           per_col=want_cols)
            stats, loss = res[0], res[1]
            per = res[2] if want_cols else None
            ev[4].record()
        else:
            stats = B.cdq_cd_solve(H, Wd, grid, scale, zero, Q, cfg.passes, ws=ws,
                                   steps_per_col=budget if args.block == 1 else None, rows16=args.rows16)
            if args.block == 2:  # the paper starts BCD from the greedy solution
                cd_stats = stats
                stats = B.cdq_bcd_solve(H, Wd, grid, scale, zero, Q, 2, budget or cfg.d_in, seed=cfg.seed, ws=ws)
                stats["cd_kernel_ms_before_bcd"] = cd_stats["kernel_ms"]
                stats["loss_after_cd"] = cd_stats["loss_after"]
            ev[4].record()
            loss = B.cdq_layer_loss(H, Wd, grid, scale, zero, Q, ws=ws, per_col=want_cols)
            if want_cols:
                loss, per = loss
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
                               ("after_cd_solve", 4, 5), ("total", 0, 5)):
                times.setdefault(name, []).append(ev[a].elapsed_time(ev[b]))
            times.setdefault("cd_kernel", []).append(stats["kernel_ms"])
            if want_cols:
                keep.update(H=H, W=Wd, scale=scale, zero=zero, Q0=Q0, Q=Q, gamma=gamma, per=per)
        if last and not host:
            # outside the step: the stand-alone loss call (the product H E on the result) for the record, and how far
            # the step's own loss is from it
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n0 = lib.cdq_kernel_launches()
            t0.record()
            ref_loss = B.cdq_layer_loss(H, Wd, grid, scale, zero, Q, ws=ws)
            t1.record()
            torch.cuda.synchronize()
            keep["untimed_launches"] = lib.cdq_kernel_launches() - n0
            keep["layer_loss_call"] = {"ms": t0.elapsed_time(t1), "loss": ref_loss,
                                       "step_loss_rel_diff": abs(loss - ref_loss) / abs(ref_loss) if ref_loss else 0.0}
        return stats, loss, d2h

    def timed(host: bool):
        for _ in range(max(warmup, 0)):
            one_step(host)
        times: dict = {}
        stats = loss = None
        d2h = 0
        multi.barrier(world)
        launches0 = lib.cdq_kernel_launches()
        for it in range(steps):
            flush.fill_(1)           # evict L2 between timed iterations (not timed)
            torch.cuda.synchronize()
            stats, loss, d2h = one_step(host, times, last=it == steps - 1)
        launches = lib.cdq_kernel_launches() - launches0 - keep.pop("untimed_launches", 0)
        multi.barrier(world)
        return times, stats, loss, d2h, launches

    def timed_stream():
        """End to end through the public streaming call (binding.quantize_layers): every step's inputs come from
        pinned host memory and its codes, scales and zeros go back to pinned host memory, all inside the timed
        region; the upload of step i + 1 runs on a second stream while step i computes (the first is not hidden)."""
        kw = {"init": args.init}
        if args.budget_div > 0:
            kw["steps_per_col"] = cfg.d_in // args.budget_div
        bufs: dict = {}
        feed = lambda k: ((Xh, Wh) for _ in range(k))
        for _ in B.quantize_layers(feed(max(warmup, 0)), grid, cfg.passes, device=dev, ws=ws, host_buffers=bufs, **kw):
            pass
        multi.barrier(world)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        d2h = 0
        for out in B.quantize_layers(feed(steps), grid, cfg.passes, device=dev, ws=ws, host_buffers=bufs, **kw):
            d2h = sum(out[k].numel() * out[k].element_size() for k in ("Q", "scale", "zero")) + 8
        t1.record()
        torch.cuda.synchronize()
        multi.barrier(world)
        return t0.elapsed_time(t1), d2h

    sampler = ClockSampler(local_rank) if (rank == 0 and sample_clocks) else None
    if sampler:
        sampler.start()
    times, stats, loss, _, launches = timed(host=False)
    clocks = sampler.stop() if sampler else None
    total_ms = sum(times["total"])
    total_ms_e2e, d2h = 0.0, 0
    streamed = args.block == 1 and not args.rows16 and not args.shard
    if e2e and streamed:
        total_ms_e2e, d2h = timed_stream()
    elif e2e:   # variants the streaming call does not cover: the same stages step by step, copies in line
        times_e2e, _, _, d2h, _ = timed(host=True)
        total_ms_e2e = sum(times_e2e["total"])
    committed = stats["committed"]
    (total_ms, total_ms_e2e), committed_all = multi.aggregate([total_ms, total_ms_e2e], committed, world, dev)
    if rank != 0:
        return None

    peaks = load_peaks()
    acc = cfg.scaled(d_out=W.shape[1], n=X.shape[0])   # what this rank worked on (the whole layer unless --shard)
    mean = lambda v: sum(v) / len(v)
    cd_ms = mean(times["cd_kernel"])
    alg_bytes = algorithmic_bytes_cd(acc, committed, 2.0 if args.rows16 else 4.0)
    if args.block == 2:  # two rows per move at most, and one H_im per pair and step
        alg_bytes += committed * 4.0 * cfg.d_in + stats["steps"] * 2.0 * cfg.d_in
    achieved = alg_bytes / (cd_ms * 1e-3) / 1e9
    h_bytes = 4.0 * cfg.d_in * cfg.d_in
    hbm_served = h_bytes > L2_BYTES
    kernel = descent_kernel_name(cfg, args.block) + ("<bf16 rows>" if args.rows16 else "")
    per_move = NCU_TRAFFIC_PER_MOVE.get((kernel, cfg.d_in))
    if hbm_served:
        roofline = {"kernel": kernel, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "frac_of_nominal_8TBs": achieved / 8000.0,
                    "traffic": per_move[0] * committed if per_move else None,
                    "traffic_source": per_move[1] if per_move else None, "algorithmic_bytes": alg_bytes,
                    "note": f"H is {h_bytes / 1e6:.0f} MB, larger than L2: rows stream from HBM; achieved = algorithmic bytes / "
                            "CUDA-event time of the descent kernel, frac of the measured HBM copy bandwidth"}
    else:
        roofline = {"kernel": kernel, "bound": "l2", "achieved": achieved, "peak": None, "unit": "GB/s", "frac": None,
                    "traffic": per_move[0] * committed if per_move else None,
                    "traffic_source": per_move[1] if per_move else None, "algorithmic_bytes": alg_bytes,
                    "note": f"H is {h_bytes / 1e6:.0f} MB and stays in L2: the rows are L2-served and the kernel is bound by "
                            "instruction issue, so `achieved` is an effective rate (algorithmic bytes / kernel time) and "
                            "no fraction of the HBM peak is claimed"}
    hess_ms = mean(times["hessian"])
    hess_flops = 2.0 * acc.n * cfg.d_in * cfg.d_in
    # flops the tensor cores actually execute: 128 x 256 tiles that touch the lower triangle
    # (tile (tm, tn) with tn <= tm // 2), over the rows padded to the 64-row K block
    tiles_m = (cfg.d_in + 127) // 128
    n_tiles = sum(tm // 2 + 1 for tm in range(tiles_m))
    tc_h = cfg.x_dtype == "bf16" and cfg.d_in >= 256
    hess_exec = 2.0 * 128 * 256 * n_tiles * ((acc.n + 63) // 64 * 64) if tc_h else hess_flops
    rec = {
        "workload": workload_name(cfg, args),
        "value": multi.whole_job_throughput(committed_all, total_ms, steps), "unit": UNIT,
        "steps": steps, "warmup": warmup, "ms_per_step": total_ms / steps, "sec_per_layer": total_ms / steps * 1e-3,
        "cd": {"committed_updates": committed, "step_budget": stats["steps"],
               "columns_converged": stats["columns_converged"], "kernel_ms": cd_ms,
               "committed_updates_per_s_kernel": committed / (cd_ms * 1e-3),
               "budget_steps_per_s_kernel": stats["steps"] / (cd_ms * 1e-3),
               "loss_before": stats["loss_before"], "loss_after": stats["loss_after"], "loss": loss,
               **({"cd_kernel_ms_before_bcd": stats["cd_kernel_ms_before_bcd"], "loss_after_cd": stats["loss_after_cd"]}
                  if args.block == 2 else {})},
        "stages_ms": {k: mean(v) for k, v in times.items()},
        # where the layer loss of the step comes from: inside cd_solve (half the dot product of the residual with the
        # descent's final gradient) or after it (the product H E)
        "loss_from": "descent gradient, inside cd_solve" if (args.block == 1 and not args.rows16) else "H E product, after cd_solve",
        "layer_loss_call": keep.get("layer_loss_call"),
        "hessian": {"ms": hess_ms, "dense_equivalent_tflops": hess_flops / (hess_ms * 1e-3) / 1e12,
                    "executed_tflops": hess_exec / (hess_ms * 1e-3) / 1e12,
                    "executed_frac_of_bf16_sustained_peak": hess_exec / (hess_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                    "executed_frac_of_bf16_burst_peak": hess_exec / (hess_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "note": "symmetric rank-k update: only lower-triangle tiles are computed; the fraction counts executed flops only"},
        "roofline": roofline,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if e2e:
        h2d = Xh.numel() * Xh.element_size() + Wh.numel() * Wh.element_size()
        rec["e2e"] = {"value": committed_all / (total_ms_e2e / steps * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": total_ms_e2e / steps,
                      "api": "binding.quantize_layers: uploads step i+1 on a second stream while step i computes; "
                             "the first upload and every download are in line; inputs (GBs) exceed L2"
                             if streamed else "stage calls with the copies in line, L2 flushed between steps"}
    if parity_cols > 0 and keep and args.block == 1 and args.init == "rtn" and args.budget_div == 0 and not args.rows16:
        rec["parity"] = parity_in_run(B, cfg, grid, keep["H"], keep["W"], keep["scale"], keep["zero"], keep["Q0"],
                                      keep["Q"], keep["gamma"], keep["per"], parity_cols)
    rec["_inputs"] = (X, W)
    return rec


def workload_name(cfg, args) -> str:
    return (f"{cfg.name}: d_in={cfg.d_in} d_out={cfg.d_out} n={cfg.n} X={cfg.x_dtype} W={cfg.w_dtype} "
            f"bits={cfg.bits} group={cfg.group_size or 'per-channel'} n_clip={cfg.n_clip} passes={cfg.passes}"
            + (" init=OWC-CD" if args.init == "owc_cd" else "")
            + (f" budget=d_in/{args.budget_div}" if args.budget_div > 0 else "")
            + (" descent=CD then BCD(k=2)" if args.block == 2 else "")
            + (" rows=bf16" if args.rows16 else ""))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="C3", choices=sorted(inputs.CONFIGS),
                    help="C3 (d_in = 14336: H exceeds L2, the descent streams its rows from HBM) is the default; C4, the largest "
                         "layer, takes ~30 s per step and is reported as a one-step record under other_configs")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the one-step records of the other benchmark layers (C1, C2, C4)")
    ap.add_argument("--oracle-cols", type=int, default=-1,
                    help="columns compared with the oracle in the run itself (default 64; 8 for C4; 0: none)")
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
    ap.add_argument("--rows16", action="store_true",
                    help="the descent reads its rows from a bf16 copy of H (cdq_cd_solve_rows16): 2 d_in bytes per move; the "
                         "reported loss is on the true H; no in-run parity (tests/test_rows16_gpu.py holds it)")
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
    profiling_case = bool(args.d_out or args.n)
    if profiling_case:
        cfg = cfg.scaled(d_out=args.d_out or cfg.d_out, n=args.n or cfg.n)
    if args.init == "owc_cd" and cfg.n_clip < 2:
        ap.error("--init owc_cd needs a config with a clipping grid (C2, C4)")

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, cfg, workload_name(cfg, args))
        return

    from paper_2406_17542_b200 import binding as B
    B.load()  # fails loudly when the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def cols_for(c):
        if args.oracle_cols >= 0:
            return args.oracle_cols
        return 0 if (profiling_case or world > 1) else (8 if c.name == "C4" else 64)

    rec = run_config(B, cfg, args, args.steps, args.warmup, dev, world, rank, e2e=True, parity_cols=cols_for(cfg),
                     sample_clocks=True, local_rank=local_rank)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    X, W = rec.pop("_inputs")
    out = {
        "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "strong" if args.shard else "weak",
        "vs_baseline": None, "dtype": "f32 scores / f64 gradient / bf16 Hessian inputs", "data": "synthetic",
        "config": {"workload": rec["workload"], "l2": "256 MiB flush between timed iterations; X also exceeds L2",
                   "per_rank": ("one layer shared out: row shards of X + one all-reduce of H, column slices of W after it"
                                if args.shard else "one independent layer per GPU, no collective")},
        "sec_per_layer": rec["sec_per_layer"], "cd": rec["cd"], "stages_ms": rec["stages_ms"], "hessian": rec["hessian"],
        "roofline": rec["roofline"], "e2e": rec["e2e"], "gpu_launches": rec["gpu_launches"], "clocks": rec["clocks"],
        "loss_from": rec["loss_from"], "layer_loss_call": rec["layer_loss_call"],
    }
    if "parity" in rec:
        out["parity"] = rec["parity"]
    if world == 1 and not args.no_cpu_baseline and args.block == 1:
        out["cpu_baseline"] = run_oracle_sample(cfg, X, W, *baseline_sample_size(cfg))
    del X, W, rec
    gc.collect()
    torch.cuda.empty_cache()
    if world == 1 and not args.no_other_configs and not profiling_case and args.block == 1 and args.init == "rtn" \
            and args.budget_div == 0 and not args.shard and not args.rows16:
        others = {}
        for name in ("C1", "C2", "C4"):
            if name == cfg.name:
                continue
            oc = inputs.CONFIGS[name]
            r = run_config(B, oc, args, 1, 1, dev, world, rank, e2e=False, parity_cols=cols_for(oc), sample_clocks=True,
                           local_rank=local_rank)
            r.pop("_inputs")
            r["note"] = "one warm-up step and one timed step"
            others[name] = r
            gc.collect()
            torch.cuda.empty_cache()
        out["other_configs"] = others
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_reference(args, cfg, workload):
    """The oracle as the timed program: each step is one bounded sample of the workload, sized from a short probe
    so that the whole run (warm-up and timed steps) takes about two and a half minutes whatever d_in and the step
    counts are: a step gets 150 s / (steps + warmup), at least 2 s and at most 20 s, half of it for the Hessian rows
    and half for grid + descent + loss of the sampled columns."""
    import oracle
    probe_rows, probe_cols = 64, 2
    X, W = inputs.make_layer(cfg.scaled(n=min(cfg.n, 8192), d_out=min(cfg.d_out, 256)), device="cpu")
    t0 = time.perf_counter()
    _, H32 = oracle.hessian(X[:probe_rows])
    rows_per_s = probe_rows / max(time.perf_counter() - t0, 1e-6)
    t0 = time.perf_counter()
    init = oracle.init_rtn(W[:, :probe_cols], cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi,
                           H=H32 if cfg.n_clip > 1 else None)
    oracle.cd_solve(H32, W[:, :probe_cols], cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in,
                    cfg.group_size)
    # columns run in parallel over the host threads: one thread's rate times the threads is what more columns get
    cols_per_s = probe_cols / max(time.perf_counter() - t0, 1e-6) * max(oracle.num_threads() // 2, 1)
    step_s = min(20.0, max(2.0, 150.0 / max(args.steps + max(args.warmup, 0), 1)))
    n_rows = int(min(X.shape[0], max(probe_rows, rows_per_s * step_s / 2)))
    n_cols = int(min(W.shape[1], max(probe_cols, cols_per_s * step_s / 2)))
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
        "config": {"workload": workload, "l2": "not applicable (host cores)",
                   "per_rank": "rank 0 only: the CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                         "sample": r["sample"] + f" (sample sized from a probe for about {step_s:.0f} s per step)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    main()
