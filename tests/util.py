"""Helpers shared by the GPU parity tests: run the oracle and the CUDA library on one layer."""
import numpy as np
import torch

import oracle
from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs


def grid_of(cfg) -> B.Grid:
    return B.Grid(cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi)


def oracle_pipeline(cfg, X, W, H32=None, lambda_rel=0.0, cols=None):
    """Oracle on the whole layer, or on a subset of its columns (columns are independent)."""
    if H32 is None:
        _, H32 = oracle.hessian(X, lambda_rel)
    Wc = W if cols is None else W[:, cols]
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi,
                           H=H32 if cfg.n_clip > 1 else None)
    res = oracle.cd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in,
                          cfg.group_size)
    total, per = oracle.layer_loss(H32, Wc, init["scale"], init["zero"], res["Q"], cfg.group_size)
    return {"H": H32, "init": init, "cd": res, "loss": total, "per_col": per}


def gpu_pipeline(cfg, X, W, mode="fast", H=None, lambda_rel=0.0, device="cuda:0"):
    """The library on the same layer.  If H is given (numpy fp32) it is used instead of cdq_hessian's."""
    Xd, Wd = X.to(device), W.to(device)
    g = grid_of(cfg)
    Hg = B.cdq_hessian(Xd, lambda_rel=lambda_rel, mode=mode)
    Huse = Hg if H is None else torch.from_numpy(np.ascontiguousarray(H)).to(device)
    scale, zero, Q0, gamma = B.cdq_init_rtn(Wd, g, H=Huse if cfg.n_clip > 1 else None, mode=mode)
    Q = Q0.clone()
    stats = B.cdq_cd_solve(Huse, Wd, g, scale, zero, Q, cfg.passes, mode=mode)
    loss, per = B.cdq_layer_loss(Huse, Wd, g, scale, zero, Q, per_col=True, mode=mode)
    torch.cuda.synchronize()
    return {"H": Hg.cpu().numpy(), "scale": scale.cpu().numpy(), "zero": zero.cpu().numpy(),
            "Q0": Q0.cpu().numpy(), "Q": Q.cpu().numpy(), "gamma": gamma.cpu().numpy(), "stats": stats,
            "loss": loss, "per_col": per.cpu().numpy(),
            "dev": {"H": Huse, "W": Wd, "grid": g, "scale": scale, "zero": zero, "Q0": Q0, "Q": Q, "gamma": gamma, "per": per}}


def check_layer_fast(cfg, ora, gpu, budget=None, label=""):
    """Whole small layer, production mode, both sides on the oracle's H: see compare_with_oracle."""
    d = gpu["dev"]
    return compare_with_oracle(cfg, ora["H"], d["H"], d["W"], np.arange(cfg.d_out), d["grid"], d["scale"], d["zero"],
                               d["Q0"], d["Q"], d["gamma"], d["per"], budget or cfg.passes * cfg.d_in, label=label)


def rel_fro(A, Bm):
    A = np.asarray(A, dtype=np.float64); Bm = np.asarray(Bm, dtype=np.float64)
    return float(np.linalg.norm(A - Bm) / np.linalg.norm(Bm))


def lib_replay(Hd, Wc_d, grid, scale_d, zero_d, Q0_d, solve=None):
    """Returns f(j, t): the library's codes of column j of the compared columns after a budget of t steps from
    Q0 (every budget is a prefix of the same deterministic trajectory).  All compared columns are re-run
    together, once per budget."""
    cache = {}

    def after(j, t):
        if t not in cache:
            Q = Q0_d.clone()
            if t > 0:
                if solve is None:
                    B.cdq_cd_solve(Hd, Wc_d, grid, scale_d, zero_d, Q, 0, steps_per_col=int(t))
                else:
                    solve(Q, int(t))
            cache[t] = Q.cpu().numpy()
        return cache[t][:, j]

    return after


def check_codes_with_fork_audit(H32, Wc, cfg, scale, zero, Q0, Q_ref, Q_lib, budget, lib_after, code_agree=0.999,
                                label=""):
    """The production-mode bar on codes: every compared column either equals the oracle's or left the oracle's
    trajectory at a step where the oracle's own gap between the two moves is below fp32 resolution
    (oracle/audit.py); over the other columns at least `code_agree` of the codes are equal.  Prints the count."""
    from oracle import audit
    Q_ref, Q_lib = np.asarray(Q_ref), np.asarray(Q_lib)
    reports = audit.audit_cd_columns(oracle, H32, Wc, cfg.bits, scale, zero, Q0, Q_ref, Q_lib, budget, cfg.group_size,
                                     lib_after)
    bad = [r for r in reports if not r["ok"]]
    forked = np.array([r["col"] for r in reports], dtype=np.int64)
    for r in reports:   # the replay must be the run that is being judged
        assert np.array_equal(lib_after(r["col"], budget), Q_lib[:, r["col"]]), ("replay differs from the run", r)
    keep = np.setdiff1d(np.arange(Q_ref.shape[1]), forked)
    agree_all = float((Q_ref == Q_lib).mean())
    agree_keep = float((Q_ref[:, keep] == Q_lib[:, keep]).mean()) if len(keep) else 1.0
    print(f"{label} columns {Q_ref.shape[1]}, forked at an fp32 near-tie {len(reports) - len(bad)}, unexplained {len(bad)}, "
          f"code agreement all {agree_all:.5f} / without audited forks {agree_keep:.5f}, "
          f"largest audited gap {max([r['gap'] for r in reports if r['ok']], default=0.0):.2e}")
    assert not bad, bad
    assert agree_keep >= code_agree, agree_keep
    return {"forks": len(reports), "agree_all": agree_all, "agree": agree_keep, "forked_cols": [r["col"] for r in reports]}


FORK_LOSS_RTOL = 0.05   # a forked column's final loss against the oracle's (another minimum of the same problem)
OWC_TIE = 1e-7   # relative gap of two clipping strengths' column losses below which the production mode's
                 # 13 slice-pair products (~1e-8 relative) may order them the other way


def compare_with_oracle(cfg, H32, Hd, Wd, cols, g, scale_d, zero_d, Q0_d, Q_d, gamma_d, per_d, budget, label="",
                        code_agree=0.999, loss_rtol=1e-4, rows16=False):
    """Production-mode result of the library on columns `cols` of a layer against the oracle on the same columns
    with the same fp32 H: grid and starting codes bit for bit, final codes up to audited fp32 near-tie forks, the
    summed column losses within loss_rtol.  With a clipping search, a column whose clipping strength differs is
    kept out of the code comparison only if the oracle's own loss table has the two strengths within OWC_TIE."""
    dev = Wd.device
    cols = np.asarray(cols)
    ct = torch.from_numpy(cols).to(dev)
    Wc = Wd[:, ct].cpu()
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, cfg.n_clip, cfg.clip_lo, cfg.clip_hi,
                           H=H32 if cfg.n_clip > 1 else None, want_loss_table=cfg.n_clip > 1)
    keep = np.arange(len(cols))
    if cfg.n_clip > 1:
        grid = oracle.gamma_grid(cfg.n_clip, cfg.clip_lo, cfg.clip_hi).astype(np.float32)
        got_gamma = gamma_d.cpu().numpy()[cols]
        same = got_gamma == grid[init["gamma_idx"]]
        for j in np.nonzero(~same)[0]:
            k_lib = int(np.argmin(np.abs(grid - got_gamma[j])))
            t = init["loss_table"][:, j]
            gap = abs(t[k_lib] - t[init["gamma_idx"][j]]) / t[init["gamma_idx"][j]]
            assert gap <= OWC_TIE, (label, "clipping strength differs at a wide gap", int(cols[j]), gap)
        print(f"{label} clipping strength differs on {int((~same).sum())} of {len(cols)} columns (all near-ties of the oracle's table)")
        keep = np.nonzero(same)[0]
    sc, ze, q0 = scale_d[:, ct].cpu().numpy(), zero_d[:, ct].cpu().numpy(), Q0_d[:, ct].cpu().numpy()
    assert np.array_equal(sc[:, keep], init["scale"][:, keep]) and np.array_equal(ze[:, keep], init["zero"][:, keep])
    assert np.array_equal(q0[:, keep], init["Q"][:, keep])
    ref = oracle.cd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], init["Q"], budget, cfg.group_size)
    _, per_ref = oracle.layer_loss(H32, Wc, init["scale"], init["zero"], ref["Q"], cfg.group_size)
    kt = ct[torch.from_numpy(keep).to(dev)]
    Wk_d, sk_d, zk_d = Wd[:, kt].contiguous(), scale_d[:, kt].contiguous(), zero_d[:, kt].contiguous()
    solve = None
    if rows16:   # the replays must be the same kind of run (Hd is then the matrix the caller handed to the library)
        solve = lambda Q, t: B.cdq_cd_solve(Hd, Wk_d, g, sk_d, zk_d, Q, 0, steps_per_col=t, rows16=True)
    replay = lib_replay(Hd, Wk_d, g, sk_d, zk_d, Q0_d[:, kt].contiguous(), solve=solve)
    Wk = Wc[:, torch.from_numpy(keep)]
    out = check_codes_with_fork_audit(H32, Wk, cfg, init["scale"][:, keep], init["zero"][:, keep], init["Q"][:, keep],
                                      ref["Q"][:, keep], Q_d[:, kt].cpu().numpy(), budget, replay, code_agree, label)
    # losses: the columns that followed the oracle's trajectory within loss_rtol; a forked column ends in another
    # coordinate-wise minimum of the same problem, a valid result whose loss differs by a percent or so
    per_got = per_d.cpu().numpy()[cols][keep]
    per_ref = per_ref[keep]
    forked = np.array(out["forked_cols"], dtype=np.int64)
    same = np.setdiff1d(np.arange(len(keep)), forked)
    assert abs(per_got[same].sum() - per_ref[same].sum()) <= loss_rtol * max(per_ref[same].sum(), 1e-30), \
        (per_got[same].sum(), per_ref[same].sum())
    if len(forked):
        assert np.all(np.abs(per_got[forked] - per_ref[forked]) <= FORK_LOSS_RTOL * per_ref[forked]), \
            (per_got[forked], per_ref[forked])
    out["gamma_mismatch"] = int(len(cols) - len(keep))
    return out


def compare_pairs_with_oracle(cfg, H32, Hd, Wd, cols, g, scale_d, zero_d, Qcd_d, Q_d, per_d, T, seed, label="",
                              code_agree=0.999, loss_rtol=1e-4, min_same_start=0.9):
    """Block descent with random pairs after the greedy descent, library against oracle on columns `cols`.  The
    two stages are judged one after the other: the pairs stage is compared on the columns whose greedy result
    is the oracle's (the others are forks of the greedy stage, which its own tests audit), from those codes."""
    from oracle import audit
    dev = Wd.device
    cols = np.asarray(cols)
    ct = torch.from_numpy(cols).to(dev)
    Wc = Wd[:, ct].cpu()
    init = oracle.init_rtn(Wc, cfg.bits, cfg.group_size, 1, 1.0, 1.0)
    cd = oracle.cd_solve(H32, Wc, cfg.bits, init["scale"], init["zero"], init["Q"], cfg.passes * cfg.d_in, cfg.group_size)
    same = (Qcd_d[:, ct].cpu().numpy() == cd["Q"]).all(axis=0)
    assert same.mean() >= min_same_start, same.mean()
    keep = np.nonzero(same)[0]
    kt = ct[torch.from_numpy(keep).to(dev)]
    Wk = Wc[:, torch.from_numpy(keep)]
    sc, ze, qs = init["scale"][:, keep], init["zero"][:, keep], cd["Q"][:, keep]
    ref = oracle.bcd_solve(H32, Wk, cfg.bits, sc, ze, qs, 2, T, seed=seed, group_size=cfg.group_size)
    Wk_d, sc_d, ze_d, qs_d = Wd[:, kt].contiguous(), scale_d[:, kt].contiguous(), zero_d[:, kt].contiguous(), Qcd_d[:, kt].contiguous()
    replay = lib_replay(Hd, Wk_d, g, sc_d, ze_d, qs_d,
                        solve=lambda Q, t: B.cdq_bcd_solve(Hd, Wk_d, g, sc_d, ze_d, Q, 2, t, seed=seed))
    got = Q_d[:, kt].cpu().numpy()
    reports = audit.audit_bcd_columns(oracle, H32, Wk, cfg.bits, sc, ze, qs, ref["Q"], got, 2, T, seed, cfg.group_size, replay)
    for r in reports:
        assert np.array_equal(replay(r["col"], T), got[:, r["col"]]), ("replay differs from the run", r)
    bad = [r for r in reports if not r["ok"]]
    forked = np.array([r["col"] for r in reports], dtype=np.int64)
    rest = np.setdiff1d(np.arange(len(keep)), forked)
    agree = float((got[:, rest] == ref["Q"][:, rest]).mean()) if len(rest) else 1.0
    print(f"{label} pairs: columns {len(keep)} (of {len(cols)} with the oracle's greedy result), forked at an fp32 near-tie "
          f"{len(reports) - len(bad)}, unexplained {len(bad)}, code agreement all {float((got == ref['Q']).mean()):.5f}, "
          f"largest audited gap {max([r['gap'] for r in reports if r['ok']], default=0.0):.2e}")
    assert not bad, bad
    assert agree >= code_agree
    per_got = per_d.cpu().numpy()[cols][keep]
    assert abs(per_got[rest].sum() - ref["loss_after"][rest].sum()) <= loss_rtol * ref["loss_after"][rest].sum()
    if len(forked):
        assert np.all(np.abs(per_got[forked] - ref["loss_after"][forked]) <= FORK_LOSS_RTOL * ref["loss_after"][forked])
    assert ref["moves"].sum() > 0 or T == 0
    return {"forks": len(reports), "agree": agree}
