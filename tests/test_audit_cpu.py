"""The fork audit (oracle/audit.py) against stand-in "libraries" whose departures from the oracle are planted
on the CPU: a departure at a wide gap must be flagged, one at an exact tie must pass, and the step found must be
the planted one."""
import numpy as np

import oracle
from oracle import audit


def _greedy(H, w, a, b, q0, L, budget, depart_at=-1, prefer_high_index=False):
    """Plain fp64 greedy descent of one column (level scan as in Algorithm 1), with a planted departure: at step
    `depart_at` it takes the second-best move; with prefer_high_index it resolves exact ties to the highest
    coordinate.  Returns the codes after every step."""
    q = q0.astype(np.int64).copy()
    states = [q.copy()]
    e = a * q + b - w
    G = 2.0 * H @ e
    hd = np.diag(H)
    for t in range(budget):
        r = np.arange(L + 1)[None, :]
        d = a * (r - q[:, None])
        delta = d * d * hd[:, None] + d * G[:, None]
        delta[np.arange(len(q)), q] = np.inf
        flat = delta.ravel()
        order = np.argsort(flat, kind="stable")
        pick = order[0]
        if flat[pick] >= 0:
            states.append(q.copy()); continue
        if prefer_high_index:
            ties = np.nonzero(flat == flat[pick])[0]
            pick = ties[-1]
        if t == depart_at:
            pick = order[1]
        i, lvl = divmod(int(pick), L + 1)
        dd = a * (lvl - q[i])
        G = G + 2.0 * dd * H[i]
        q[i] = lvl
        states.append(q.copy())
    return states


def _layer(seed, d_in=24, n=96, duplicate=False):
    rng = np.random.default_rng(seed)
    X = rng.normal(size=(n, d_in)).astype(np.float32)
    w = rng.normal(size=d_in) * 0.02
    if duplicate:      # two identical features with identical weights: their moves tie exactly
        X[:, 2] *= 3.0
        X[:, 5] = X[:, 2]
        w[5] = w[2]
    _, H32 = oracle.hessian(X)
    return H32, w.astype(np.float32)


def _run(H32, w, bits, budget, scramble=True, **planted):
    W = w.reshape(-1, 1)
    init = oracle.init_rtn(W, bits)
    if scramble:   # start far from a coordinate-wise minimum, so that the descent has many moves to make
        init["Q"] = np.random.default_rng(5).integers(0, 1 << bits, size=init["Q"].shape).astype(np.uint8)
        init["Q"][5] = init["Q"][2]   # (only matters for the layer with two identical features)
    ref = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], budget, 0)
    L = (1 << bits) - 1
    d_in = len(w)
    a = audit.expand(init["scale"][:, 0], d_in, 0)
    b = audit.expand(init["zero"][:, 0], d_in, 0)
    states = _greedy(H32.astype(np.float64), w.astype(np.float64), a[0], b[0], init["Q"][:, 0], L, budget, **planted)
    lib_after = lambda j, t: states[t]
    Q_lib = states[budget].astype(np.uint8).reshape(-1, 1)
    return audit.audit_cd_columns(oracle, H32, W, bits, init["scale"], init["zero"], init["Q"], ref["Q"], Q_lib, budget, 0,
                                  lib_after), ref, Q_lib


def test_stand_in_that_follows_the_oracle_has_nothing_to_audit():
    H32, w = _layer(0)
    reports, ref, Q_lib = _run(H32, w, 3, 24)
    assert np.array_equal(ref["Q"], Q_lib) and reports == []


def test_departure_at_a_wide_gap_is_flagged_at_its_step():
    H32, w = _layer(1)
    reports, ref, Q_lib = _run(H32, w, 3, 4, depart_at=3)   # the budget ends at the planted step: the codes differ
    assert len(reports) == 1
    r = reports[0]
    assert r["step"] == 4 and not r["ok"] and r["gap"] > 1e-4
    assert r["delta_ref"] < r["delta_lib"] < 0       # the oracle's move is the better one


def test_exact_tie_resolved_the_other_way_passes():
    H32, w = _layer(2, duplicate=True)
    reports, ref, Q_lib = _run(H32, w, 3, 2, prefer_high_index=True)
    assert len(reports) == 1                         # coordinate 5 moved where the oracle moved coordinate 2
    assert ref["Q"][2, 0] != Q_lib[2, 0] and ref["Q"][5, 0] != Q_lib[5, 0]
    assert reports[0]["ok"] and reports[0]["gap"] <= 1e-12
