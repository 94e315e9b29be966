"""Fork audit for the production-mode parity tests (test infrastructure, like the rest of oracle/).

The production kernels score moves in fp32.  Greedy picks are discrete, so when the two best moves
of a step are closer than fp32 resolves, the library may take the other one; from there its
trajectory and the oracle's differ ("fork"), and a tenth of the column's codes may end up different
although both results are valid runs of the algorithm (Algorithm 1 fixes no arithmetic).

This module decides whether a column that differs is such a fork.  It never looks inside the
library: the caller passes a function that runs the library on that one column with a step budget
t and returns its codes.  Budgets are prefixes of one deterministic trajectory, so bisection over t
finds the first step t* at which the library leaves the oracle's trajectory; both sides share the
state before it.  The audit then evaluates, in fp64 from the definition of the loss change
(delta^T H delta + delta^T G with G = 2 H (w_hat - w), the identity below Algorithm 1), the move the
oracle took and the move the library took at t*, and reports the gap between them relative to the
magnitude of the terms of the oracle's move.  A fork is legitimate when that gap is below what fp32
scores can resolve.
"""
from __future__ import annotations

import numpy as np

# fp32 scoring: the gradient rounded to fp32 (2^-24), one fused multiply-add and one product (2^-24
# each), on terms d^2 H_ii and d g_i that cancel by a factor of up to ~2 in the sum; 2^-21 covers it.
FP32_GAP = 2.0 ** -21


def _states_from_trace(q0, trace_i, trace_r):
    """Returns a function t -> codes after t moves that replays incrementally (bisection calls it out of order)."""
    cache = {0: np.array(q0, dtype=np.int64, copy=True)}

    def after(t: int) -> np.ndarray:
        t = min(int(t), len(trace_i))
        if t in cache:
            return cache[t]
        base = max(k for k in cache if k <= t)
        q = cache[base].copy()
        for s in range(base, t):
            q[trace_i[s]] = trace_r[s]
        cache[t] = q
        return q

    return after


def move_change(H32: np.ndarray, w: np.ndarray, a_full: np.ndarray, b_full: np.ndarray, q_prev: np.ndarray,
                q_next: np.ndarray):
    """Change of the column loss for the move q_prev -> q_next, in fp64 from its definition, and the sum
    of the magnitudes of its terms.  a_full, b_full: scale and zero of every coordinate."""
    S = np.nonzero(q_next != q_prev)[0]
    if len(S) == 0:
        return 0.0, 0.0
    e = a_full * q_prev.astype(np.float64) + b_full - w
    rows = H32[S, :].astype(np.float64)
    G = 2.0 * (rows @ e)
    d = a_full[S] * (q_next[S] - q_prev[S]).astype(np.float64)
    HSS = rows[:, S]
    quad = float(d @ HSS @ d)
    lin = d * G
    mag = float(np.abs(np.outer(d, d) * HSS).sum() + np.abs(lin).sum())
    return quad + float(lin.sum()), mag


def audit_column(H32, w, a_full, b_full, q0, ref_after, lib_after, budget: int, tol: float = FP32_GAP) -> dict:
    """Audits one column whose final codes differ.

    ref_after(t), lib_after(t): codes [d_in] after a budget of t steps from q0, oracle and library.
    Returns {"step": t*, "gap": relative gap, "ok": gap <= tol, "delta_ref", "delta_lib"}."""
    lo, hi = 0, int(budget)          # invariant: equal at lo, different at hi
    if np.array_equal(ref_after(hi), lib_after(hi)):   # the replay does not differ: nothing to audit, and nothing explained
        return {"step": -1, "gap": float("inf"), "ok": False, "delta_ref": 0.0, "delta_lib": 0.0}
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if np.array_equal(ref_after(mid), lib_after(mid)):
            lo = mid
        else:
            hi = mid
    q_prev = ref_after(lo).astype(np.int64)
    d_ref, mag_ref = move_change(H32, w, a_full, b_full, q_prev, ref_after(hi).astype(np.int64))
    d_lib, mag_lib = move_change(H32, w, a_full, b_full, q_prev, lib_after(hi).astype(np.int64))
    scale = max(mag_ref, mag_lib, 1e-300)
    gap = abs(d_ref - d_lib) / scale
    return {"step": hi, "gap": gap, "ok": bool(gap <= tol), "delta_ref": d_ref, "delta_lib": d_lib}


def expand(v, d_in: int, group_size: int) -> np.ndarray:
    """Per-group values [d_in/g] of one column -> per-coordinate [d_in] fp64."""
    v = np.asarray(v, dtype=np.float64).reshape(-1)
    g = group_size if group_size else d_in
    return np.repeat(v, g)[:d_in]


def audit_cd_columns(oracle_mod, H32, Wc, bits, scale, zero, Q0, Q_ref, Q_lib, budget, group_size, lib_after_col,
                     tol: float = FP32_GAP) -> list:
    """Audits every column of a greedy-descent comparison whose library codes differ from the oracle's.

    Wc, scale, zero, Q0, Q_ref, Q_lib: the compared columns (arrays with one column per problem);
    lib_after_col(j, t): the library's codes of compared column j after a budget of t steps.
    The oracle's trajectory comes from its own trace of that column."""
    out = []
    Wn = oracle_mod._f64(Wc)
    d_in = Wn.shape[0]
    for j in np.nonzero((np.asarray(Q_ref) != np.asarray(Q_lib)).any(axis=0))[0]:
        j = int(j)
        res = oracle_mod.cd_solve(H32, Wn[:, j:j + 1], bits, np.asarray(scale)[:, j:j + 1], np.asarray(zero)[:, j:j + 1],
                                  np.asarray(Q0)[:, j:j + 1], budget, group_size, trace_col=0)
        tr = res["trace"]
        ref_after = _states_from_trace(np.asarray(Q0)[:, j], tr["i"], tr["r"])
        cache = {}

        def lib_after(t, j=j, cache=cache):
            if t not in cache:
                cache[t] = np.asarray(lib_after_col(j, int(t)), dtype=np.int64)
            return cache[t]

        r = audit_column(H32, Wn[:, j], expand(np.asarray(scale)[:, j], d_in, group_size),
                         expand(np.asarray(zero)[:, j], d_in, group_size), np.asarray(Q0)[:, j], ref_after, lib_after,
                         budget, tol)
        r["col"] = j
        out.append(r)
    return out


def audit_bcd_columns(oracle_mod, H32, Wc, bits, scale, zero, Qstart, Q_ref, Q_lib, k, budget, seed, group_size,
                      lib_after_col, tol: float = FP32_GAP) -> list:
    """The same audit for block coordinate descent with random blocks (Algorithm 2 / 5) from the codes Qstart.
    The oracle has no trace for it; its state after t steps is a run with budget t (the partition of a step
    depends on the step and the seed only, so budgets are prefixes of one trajectory here too)."""
    out = []
    Wn = oracle_mod._f64(Wc)
    d_in = Wn.shape[0]
    for j in np.nonzero((np.asarray(Q_ref) != np.asarray(Q_lib)).any(axis=0))[0]:
        j = int(j)
        sc, ze, qs = np.asarray(scale)[:, j:j + 1], np.asarray(zero)[:, j:j + 1], np.asarray(Qstart)[:, j:j + 1]
        rcache, lcache = {0: qs[:, 0].astype(np.int64)}, {}

        def ref_after(t, rcache=rcache, sc=sc, ze=ze, qs=qs, j=j):
            if t not in rcache:
                r = oracle_mod.bcd_solve(H32, Wn[:, j:j + 1], bits, sc, ze, qs, k, int(t), seed=seed, group_size=group_size)
                rcache[t] = r["Q"][:, 0].astype(np.int64)
            return rcache[t]

        def lib_after(t, j=j, lcache=lcache):
            if t not in lcache:
                lcache[t] = np.asarray(lib_after_col(j, int(t)), dtype=np.int64)
            return lcache[t]

        r = audit_column(H32, Wn[:, j], expand(sc[:, 0], d_in, group_size), expand(ze[:, 0], d_in, group_size), qs[:, 0],
                         ref_after, lib_after, budget, tol)
        r["col"] = j
        out.append(r)
    return out
