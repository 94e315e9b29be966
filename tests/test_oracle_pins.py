"""Pins for the fp64 CPU oracle: checks against what the paper and the mathematics fix,
none of which go through the oracle's own formulas.

Each test names the passage it pins.  The direct loss ||X (w - w_hat)||^2 is always
computed here from X with numpy, never from H.
"""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _layer(seed, n, d_in, d_out, feat_sigma=1.0, w_sigma=0.02):
    rng = np.random.default_rng(seed)
    s = np.exp(feat_sigma * rng.standard_normal(d_in))
    X = (rng.standard_normal((n, d_in)) * s).astype(np.float32)
    W = (w_sigma * rng.standard_normal((d_in, d_out))).astype(np.float32)
    return X, W


def _expand(v, d_in):
    """[d_in/g, d_out] -> [d_in, d_out]."""
    g = d_in // v.shape[0]
    return np.repeat(v.astype(np.float64), g, axis=0)


def _direct_loss(X, W, scale, zero, Q):
    """sum_j ||X (w_j - a q_j - b)||^2 straight from X (Eq. 1)."""
    d_in = W.shape[0]
    What = _expand(scale, d_in) * Q.astype(np.float64) + _expand(zero, d_in)
    R = X.astype(np.float64) @ (W.astype(np.float64) - What)
    return (R * R).sum(axis=0)


# ---------------------------------------------------------------- Hessian
def test_hessian_matches_blas_and_is_symmetric():
    X, _ = _layer(1, 300, 37, 1)
    H64, H32 = oracle.hessian(X)
    ref = X.astype(np.float64).T @ X.astype(np.float64)
    np.testing.assert_allclose(H64, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())
    assert np.array_equal(H64, H64.T)
    assert np.array_equal(H32, H64.astype(np.float32))


def test_hessian_lambda_adds_scaled_mean_diagonal():
    X, _ = _layer(2, 64, 16, 1)
    H0, _ = oracle.hessian(X)
    H1, _ = oracle.hessian(X, lambda_rel=0.25)
    D = H1 - H0
    assert np.allclose(D - np.diag(np.diag(D)), 0.0)
    np.testing.assert_allclose(np.diag(D), 0.25 * np.trace(H0) / 16, rtol=1e-12)


def test_hessian_entries_match_full():
    X, _ = _layer(3, 200, 23, 1)
    H64, _ = oracle.hessian(X)
    rows = np.array([0, 5, 22, 7]); cols = np.array([0, 9, 22, 3])
    np.testing.assert_allclose(oracle.hessian_entries(X, rows, cols), H64[rows, cols], rtol=1e-13)


# ---------------------------------------------------------------- Eq. 2
def _read_cols(name):
    rows = [l.split() for l in open(os.path.join(GOLD, name)) if l.strip() and not l.startswith("#")]
    return np.array(rows, dtype=np.float64)


def test_rtn_hand_worked_half_to_even():
    t = _read_cols("rtn_half_even.txt")
    out = oracle.init_rtn(t[:, :1], bits=2)
    assert out["scale"][0, 0] == 1.0 and out["zero"][0, 0] == -1.0
    assert out["Q"][:, 0].tolist() == t[:, 1].astype(int).tolist()


def test_owc_hand_worked_clip():
    t = _read_cols("owc_clip_by_hand.txt")
    H = np.eye(7, dtype=np.float32)
    # a one-point grid at 0.5 is not expressible (one point => MinMax), so use {0.5, 0.5}
    out = oracle.init_rtn(t[:, :1], bits=2, n_clip=2, clip_lo=0.5, clip_hi=0.5, H=H, want_loss_table=True)
    assert out["scale"][0, 0] == 0.5 and out["zero"][0, 0] == -1.0
    assert out["Q"][:, 0].tolist() == t[:, 1].astype(int).tolist()
    what = 0.5 * out["Q"][:, 0] - 1.0
    assert what.tolist() == t[:, 2].tolist()
    # with H = I the loss is the squared error of the hand-worked w_hat
    np.testing.assert_allclose(out["loss_table"][0, 0], ((t[:, 0] - t[:, 2]) ** 2).sum(), rtol=1e-14)


@pytest.mark.parametrize("bits,g", [(2, 0), (3, 8), (4, 16)])
def test_gamma_one_is_minmax_and_codes_are_nearest_levels(bits, g):
    _, W = _layer(4, 8, 32, 5)
    out = oracle.init_rtn(W, bits=bits, group_size=g)
    L = 2 ** bits - 1
    gg = g or 32
    Wg = W.reshape(32 // gg, gg, 5).astype(np.float64)
    mn, mx = Wg.min(axis=1), Wg.max(axis=1)
    assert np.array_equal(out["zero"], mn.astype(np.float32))
    assert np.array_equal(out["scale"], ((mx - mn) / L).astype(np.float32))
    # every code is a nearest level: |w - (a q + b)| <= a/2 (+ulp) inside the grid
    a = _expand(out["scale"], 32); b = _expand(out["zero"], 32)
    err = np.abs(W - (a * out["Q"] + b))
    assert (err <= a / 2 * (1 + 1e-6)).all()
    assert out["Q"].max() <= L


def test_owc_never_worse_than_minmax_and_table_matches_direct_loss():
    X, W = _layer(5, 96, 24, 6)
    _, H32 = oracle.hessian(X)
    mm = oracle.init_rtn(W, bits=3, group_size=8)
    ow = oracle.init_rtn(W, bits=3, group_size=8, n_clip=6, clip_lo=0.5, clip_hi=1.0, H=H32,
                         want_loss_table=True)
    _, per_mm = oracle.layer_loss(H32, W, mm["scale"], mm["zero"], mm["Q"], group_size=8)
    _, per_ow = oracle.layer_loss(H32, W, ow["scale"], ow["zero"], ow["Q"], group_size=8)
    assert (per_ow <= per_mm).all()
    # the last grid point is gamma = 1 == MinMax
    np.testing.assert_allclose(ow["loss_table"][-1], per_mm, rtol=1e-12)
    # chosen entry is the column minimum, lowest index on ties
    assert np.array_equal(ow["gamma_idx"], ow["loss_table"].argmin(axis=0))
    # the table agrees with the loss recomputed from X for one re-derived gamma
    k = 2
    gam = 0.5 + 0.5 * k / 5
    Wg = W.reshape(3, 8, 6).astype(np.float64)
    mn, mx = Wg.min(axis=1), Wg.max(axis=1)
    a = (gam * (mx - mn) / 7).astype(np.float32)
    Q = np.clip(np.rint((Wg - mn[:, None]) / a.astype(np.float64)[:, None]), 0, 7).reshape(24, 6)
    direct = _direct_loss(X, W, a, mn.astype(np.float32), Q)
    np.testing.assert_allclose(ow["loss_table"][k], direct, rtol=2e-5)  # H was rounded to fp32


# ---------------------------------------------------------------- greedy CD
def _setup(seed, n, d_in, d_out, bits, g=0, **kw):
    X, W = _layer(seed, n, d_in, d_out, **kw)
    _, H32 = oracle.hessian(X)
    init = oracle.init_rtn(W, bits=bits, group_size=g)
    return X, W, H32, init


def test_layer_loss_equals_direct_loss_from_x():
    X, W, H32, init = _setup(6, 128, 20, 7, 3, g=5)
    tot, per = oracle.layer_loss(H32, W, init["scale"], init["zero"], init["Q"], group_size=5)
    direct = _direct_loss(X, W, init["scale"], init["zero"], init["Q"])
    np.testing.assert_allclose(per, direct, rtol=2e-5)
    np.testing.assert_allclose(tot, direct.sum(), rtol=2e-5)


@pytest.mark.parametrize("bits,g", [(2, 0), (3, 0), (4, 0), (2, 4), (3, 8)])
def test_delta_identity_and_monotone_loss(bits, g):
    """Section 3.1: the printed decrease equals the change of the loss, recomputed from X."""
    d_in = 16
    X, W, H32, init = _setup(7 + bits, 64, d_in, 3, bits, g=g)
    # use the exactly representable H (fp32) on both sides: rebuild X-loss via H64 of fp32 H
    col = 1
    res = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], steps_per_col=3 * d_in,
                          group_size=g, trace_col=col)
    tr = res["trace"]
    assert len(tr["i"]) > 0
    assert (tr["delta"] < 0).all()                       # strictly improving moves only
    H = H32.astype(np.float64)
    a = _expand(init["scale"], d_in)[:, col]; b = _expand(init["zero"], d_in)[:, col]
    w = W[:, col].astype(np.float64)
    q = init["Q"][:, col].astype(np.float64)
    def loss(qv):
        e = a * qv + b - w
        return e @ H @ e
    cur = loss(q)
    for i, r, dlt in zip(tr["i"], tr["r"], tr["delta"]):
        q2 = q.copy(); q2[i] = r
        new = loss(q2)
        assert abs((new - cur) - dlt) <= 1e-9 * max(abs(cur), 1e-30)
        assert new < cur
        q, cur = q2, new
    assert np.array_equal(q.astype(np.uint8), res["Q"][:, col])


def test_delta_matches_loss_change_recomputed_from_x():
    """Same identity, with the loss taken straight from X (no H) for the first moves."""
    d_in = 12
    X, W, H32, init = _setup(21, 48, d_in, 2, 3)
    res = oracle.cd_solve(H32, W, 3, init["scale"], init["zero"], init["Q"], steps_per_col=d_in, trace_col=0)
    Q = init["Q"].copy()
    cur = _direct_loss(X, W, init["scale"], init["zero"], Q)[0]
    for i, r, dlt in zip(res["trace"]["i"], res["trace"]["r"], res["trace"]["delta"]):
        Q[i, 0] = r
        new = _direct_loss(X, W, init["scale"], init["zero"], Q)[0]
        assert abs((new - cur) - dlt) <= 3e-5 * abs(cur)   # fp32 rounding of H only
        cur = new


def test_incremental_gradient_equals_fresh_gradient():
    d_in, d_out = 40, 6
    X, W, H32, init = _setup(8, 160, d_in, d_out, 4, g=8)
    res = oracle.cd_solve(H32, W, 4, init["scale"], init["zero"], init["Q"], steps_per_col=2 * d_in,
                          group_size=8, want_G=True)
    assert res["committed"] > 0
    What = _expand(init["scale"], d_in) * res["Q"] + _expand(init["zero"], d_in)
    fresh = (2.0 * H32.astype(np.float64) @ (What - W.astype(np.float64))).T
    scale = np.abs(fresh).max()
    assert np.abs(res["G"] - fresh).max() <= 1e-9 * scale
    # and the oracle's own fresh gradient routine agrees with the numpy one
    G2 = oracle.gradient(H32, W, init["scale"], init["zero"], res["Q"], group_size=8)
    assert np.abs(G2 - fresh).max() <= 1e-12 * scale


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_first_pick_equals_closed_form_coordinate_optimum(bits):
    """The best level of a coordinate is the clamped rounding of the parabola's vertex."""
    d_in = 24
    X, W, H32, init = _setup(30 + bits, 100, d_in, 4, bits)
    L = 2 ** bits - 1
    G = oracle.gradient(H32, W, init["scale"], init["zero"], init["Q"])
    for col in range(4):
        res = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], steps_per_col=1,
                              trace_col=col)
        a = float(init["scale"][0, col]); q = init["Q"][:, col].astype(np.float64)
        hd = np.diag(H32).astype(np.float64); g = G[col]
        vertex = q - g / (2 * a * hd)
        best = (0.0, -1, -1)
        for i in range(d_in):
            for r in {int(np.clip(np.floor(vertex[i]), 0, L)), int(np.clip(np.ceil(vertex[i]), 0, L))}:
                d = a * (r - q[i])
                dl = d * d * hd[i] + d * g[i]
                if dl < best[0] - 1e-15 * abs(best[0]):
                    best = (dl, i, r)
        if res["moves_per_col"][col] == 0:
            assert best[1] == -1
        else:
            assert (res["trace"]["i"][0], res["trace"]["r"][0]) == (best[1], best[2])
            np.testing.assert_allclose(res["trace"]["delta"][0], best[0], rtol=1e-12)


def test_brute_force_optimum_bounds_greedy():
    """Eq. 1 for fixed (a, b) is integer least squares: exact <= greedy <= round-to-nearest."""
    for seed in range(4):
        d_in, bits = 6 + seed % 3, 2
        X, W, H32, init = _setup(40 + seed, 4 * d_in, d_in, 3, bits, feat_sigma=0.7)
        res = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], steps_per_col=50 * d_in)
        _, per_init = oracle.layer_loss(H32, W, init["scale"], init["zero"], init["Q"])
        _, per_cd = oracle.layer_loss(H32, W, init["scale"], init["zero"], res["Q"])
        H = H32.astype(np.float64)
        codes = np.array(list(itertools.product(range(4), repeat=d_in)), dtype=np.float64)
        for col in range(3):
            a = float(init["scale"][0, col]); b = float(init["zero"][0, col])
            E = a * codes + b - W[:, col].astype(np.float64)
            losses = np.einsum("ci,ij,cj->c", E, H, E)
            exact = losses.min()
            assert exact <= per_cd[col] * (1 + 1e-12)
            assert per_cd[col] <= per_init[col] * (1 + 1e-12)
            # greedy ends in a point no single-coordinate change improves
            qcd = res["Q"][:, col]
            idx = int(sum(int(v) * 4 ** (d_in - 1 - k) for k, v in enumerate(qcd)))
            np.testing.assert_allclose(losses[idx], per_cd[col], rtol=1e-10)


def test_diagonal_hessian_needs_no_move():
    """Separable problem: round-to-nearest with clamping is already optimal."""
    rng = np.random.default_rng(50)
    d_in = 32
    H = np.diag(rng.uniform(0.5, 3.0, d_in)).astype(np.float32)
    W = (0.02 * rng.standard_normal((d_in, 4))).astype(np.float32)
    init = oracle.init_rtn(W, bits=3, group_size=8)
    res = oracle.cd_solve(H, W, 3, init["scale"], init["zero"], init["Q"], steps_per_col=d_in, group_size=8)
    assert res["committed"] == 0 and res["columns_converged"] == 4
    assert np.array_equal(res["Q"], init["Q"])


def test_single_coordinate_reduces_to_nearest_level():
    H = np.array([[2.5]], dtype=np.float32)
    W = np.array([[0.3, -0.7, 0.11]], dtype=np.float32)
    a = np.full((1, 3), 0.1, dtype=np.float32); b = np.full((1, 3), -0.8, dtype=np.float32)
    Q0 = np.array([[0, 15, 7]], dtype=np.uint8)            # deliberately wrong starts
    res = oracle.cd_solve(H, W, 4, a, b, Q0, steps_per_col=4)
    want = np.clip(np.rint((W.astype(np.float64) - (-0.8)) / 0.1), 0, 15).astype(np.uint8)
    assert np.array_equal(res["Q"], want)
    assert (res["moves_per_col"] <= 1).all()               # one move reaches the best level


@pytest.mark.parametrize("g", [0, 4])
def test_code_unit_algorithm_picks_same_moves(g):
    """Algorithm 4 (Algorithm 1 when the scale is constant) == the weight-unit iteration."""
    d_in = 16
    X, W, H32, init = _setup(60 + g, 80, d_in, 3, 3, g=g)
    for col in range(3):
        res = oracle.cd_solve(H32, W, 3, init["scale"], init["zero"], init["Q"], steps_per_col=2 * d_in,
                              group_size=g, trace_col=col)
        a = _expand(init["scale"], d_in)[:, col]; b = _expand(init["zero"], d_in)[:, col]
        lit = oracle.cd_code_units(H32, W[:, col], a, b, 3, init["Q"][:, col], 2 * d_in)
        assert lit["moves"] == res["moves_per_col"][col]
        assert np.array_equal(lit["trace_i"], res["trace"]["i"])
        assert np.array_equal(lit["trace_r"], res["trace"]["r"])
        assert np.array_equal(lit["q"], res["Q"][:, col])


def test_converged_point_is_coordinatewise_optimal():
    d_in, bits = 20, 3
    X, W, H32, init = _setup(70, 100, d_in, 5, bits)
    res = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], steps_per_col=100 * d_in)
    assert res["columns_converged"] == 5
    H = H32.astype(np.float64)
    for col in range(5):
        a = float(init["scale"][0, col]); b = float(init["zero"][0, col])
        w = W[:, col].astype(np.float64); q = res["Q"][:, col].astype(np.float64)
        base = (a * q + b - w) @ H @ (a * q + b - w)
        for i in range(d_in):
            for r in range(2 ** bits):
                q2 = q.copy(); q2[i] = r
                e = a * q2 + b - w
                assert e @ H @ e >= base * (1 - 1e-12)


def test_step_budget_is_respected_and_stats_consistent():
    d_in = 24
    X, W, H32, init = _setup(80, 100, d_in, 8, 4)
    full = oracle.cd_solve(H32, W, 4, init["scale"], init["zero"], init["Q"], steps_per_col=100 * d_in)
    cut = oracle.cd_solve(H32, W, 4, init["scale"], init["zero"], init["Q"], steps_per_col=3)
    assert (cut["moves_per_col"] <= 3).all()
    assert cut["steps"] == 3 * 8 and cut["committed"] == cut["moves_per_col"].sum()
    assert full["loss_after"] <= cut["loss_after"] <= cut["loss_before"] == full["loss_before"]
    # resuming the cut run reaches the same point as the uninterrupted run
    rest = oracle.cd_solve(H32, W, 4, init["scale"], init["zero"], cut["Q"], steps_per_col=100 * d_in)
    assert np.array_equal(rest["Q"], full["Q"])


def test_tie_break_lowest_coordinate_then_lowest_level():
    """Two identical, uncoupled coordinates with the vertex half way between two levels."""
    H = np.diag([1.0, 1.0]).astype(np.float32)
    a = np.array([[1.0]], dtype=np.float32); b = np.array([[0.0]], dtype=np.float32)
    W = np.array([[2.0], [2.0]], dtype=np.float32)
    Q0 = np.array([[0], [0]], dtype=np.uint8)              # both want level 2; Delta equal
    res = oracle.cd_solve(H, W, 2, a, b, Q0, steps_per_col=1, trace_col=0)
    assert (res["trace"]["i"][0], res["trace"]["r"][0]) == (0, 2)
    W2 = np.array([[1.5], [0.0]], dtype=np.float32)        # levels 1 and 2 tie for coordinate 0
    res = oracle.cd_solve(H, W2, 2, a, b, Q0, steps_per_col=1, trace_col=0)
    assert (res["trace"]["i"][0], res["trace"]["r"][0]) == (0, 1)


# ---------------------------------------------------------------- OWC-CD (Algorithm 3)
def _group_grids(W, H32, bits, g, grid):
    """Per group t and grid point k: (a, b, q) of Eq. 2 for every column, from the pinned per-channel
    routine on the group's rows (a two-point grid with both points at gamma_k forces that gamma)."""
    d_in, d_out = W.shape
    out = {}
    for t in range(d_in // g):
        rows = slice(t * g, (t + 1) * g)
        Hs = np.ascontiguousarray(H32[rows, rows])
        for k, gam in enumerate(grid):
            r = oracle.init_rtn(W[rows], bits, 0, n_clip=2, clip_lo=float(gam), clip_hi=float(gam), H=Hs)
            out[(t, k)] = (r["scale"][0], r["zero"][0], r["Q"])
    return out


def _assemble(grids, choice, d_in, d_out, g):
    """Layer grid and codes when group t of column j uses grid point choice[t, j]."""
    ng = d_in // g
    scale = np.empty((ng, d_out), np.float32); zero = np.empty((ng, d_out), np.float32)
    Q = np.empty((d_in, d_out), np.uint8)
    for t in range(ng):
        for j in range(d_out):
            a, b, q = grids[(t, int(choice[t, j]))]
            scale[t, j] = a[j]; zero[t, j] = b[j]; Q[t * g:(t + 1) * g, j] = q[:, j]
    return scale, zero, Q


def test_owc_cd_tracked_loss_is_the_loss_from_x_and_never_rises():
    d_in, d_out, g, bits = 32, 6, 8, 3
    X, W = _layer(41, 200, d_in, d_out, feat_sigma=1.2)
    _, H32 = oracle.hessian(X)
    for steps in (0, 1, 2, d_in // g, 50):
        r = oracle.owc_cd(H32, W, bits, g, 6, 0.5, 1.0, steps)
        direct = _direct_loss(X, W, r["scale"], r["zero"], r["Q"])
        # the running loss (start + predicted changes) is the loss recomputed from X: pins the
        # sign and the factor 2 of the linear term and the block of H in the quadratic term
        np.testing.assert_allclose(r["loss_after"], direct, rtol=1e-5)      # H is fp32: X^T X rounded
        _, per = oracle.layer_loss(H32, W, r["scale"], r["zero"], r["Q"], g)
        np.testing.assert_allclose(r["loss_after"], per, rtol=1e-10)
        assert (r["loss_after"] <= r["loss_before"]).all() and (r["moves"] <= steps).all()
    # step 0 is MinMax when the grid ends at 1
    r0 = oracle.owc_cd(H32, W, bits, g, 6, 0.5, 1.0, 0)
    mm = oracle.init_rtn(W, bits, g)
    assert np.array_equal(r0["Q"], mm["Q"]) and np.array_equal(r0["scale"], mm["scale"])


def test_owc_cd_with_one_group_is_the_owc_grid_search():
    d_in, d_out, bits = 16, 12, 3
    X, W = _layer(42, 120, d_in, d_out)
    _, H32 = oracle.hessian(X)
    owc = oracle.init_rtn(W, bits, 0, n_clip=8, clip_lo=0.4, clip_hi=1.0, H=H32, want_loss_table=True)
    r = oracle.owc_cd(H32, W, bits, 0, 8, 0.4, 1.0, 1)
    # one change from the last grid point lands on the grid search's minimiser
    assert np.array_equal(r["gamma_idx"][0], owc["gamma_idx"])
    assert np.array_equal(r["Q"], owc["Q"]) and np.array_equal(r["scale"], owc["scale"])
    np.testing.assert_allclose(r["loss_after"], owc["loss_table"].min(axis=0), rtol=1e-10)


def test_owc_cd_against_brute_force_over_all_assignments():
    d_in, d_out, g, bits, nk = 12, 5, 4, 2, 4
    X, W = _layer(43, 90, d_in, d_out, feat_sigma=1.0)
    _, H32 = oracle.hessian(X)
    grid = oracle.gamma_grid(nk, 0.5, 1.0)
    grids = _group_grids(W, H32, bits, g, grid)
    ng = d_in // g
    losses = {}
    for combo in itertools.product(range(nk), repeat=ng):
        choice = np.repeat(np.array(combo)[:, None], d_out, axis=1)
        s, z, Q = _assemble(grids, choice, d_in, d_out, g)
        losses[combo] = oracle.layer_loss(H32, W, s, z, Q, g)[1]
    exact = np.min(np.stack(list(losses.values())), axis=0)
    start = losses[(nk - 1,) * ng]
    r = oracle.owc_cd(H32, W, bits, g, nk, 0.5, 1.0, 100)
    assert (exact <= r["loss_after"] * (1 + 1e-12)).all() and (r["loss_after"] <= start * (1 + 1e-12)).all()
    for j in range(d_out):
        combo = tuple(int(v) for v in r["gamma_idx"][:, j])
        np.testing.assert_allclose(r["loss_after"][j], losses[combo][j], rtol=1e-10)
        # converged: no single group change lowers the loss
        for t in range(ng):
            for k in range(nk):
                other = combo[:t] + (k,) + combo[t + 1:]
                assert losses[other][j] >= losses[combo][j] * (1 - 1e-12)
    # the first change is the best single-group change from the start
    r1 = oracle.owc_cd(H32, W, bits, g, nk, 0.5, 1.0, 1)
    for j in range(d_out):
        singles = {(t, k): losses[tuple(k if u == t else nk - 1 for u in range(ng))][j]
                   for t in range(ng) for k in range(nk - 1)}
        (bt, bk), bl = min(singles.items(), key=lambda kv: (kv[1], kv[0]))
        if bl < start[j]:
            assert r1["moves"][j] == 1 and int(r1["gamma_idx"][bt, j]) == bk
        else:
            assert r1["moves"][j] == 0


# ---------------------------------------------------------------- BCD with random blocks (Algorithm 2 / 5)
def test_bcd_partition_is_a_permutation_and_varies():
    for d in (1, 2, 7, 10, 64, 100, 257):
        p0 = oracle.bcd_perm(d, 11, 0)
        assert sorted(p0.tolist()) == list(range(d))
        if d >= 10:
            assert not np.array_equal(p0, oracle.bcd_perm(d, 11, 1))      # another step
            assert not np.array_equal(p0, oracle.bcd_perm(d, 12, 0))      # another seed
    # every pair of coordinates gets paired at some step: the family is not stuck on a few partitions
    d, seen = 12, set()
    for t in range(400):
        p = oracle.bcd_perm(d, 5, t)
        seen |= {tuple(sorted((int(p[2 * u]), int(p[2 * u + 1])))) for u in range(d // 2)}
    assert len(seen) == d * (d - 1) // 2


@pytest.mark.parametrize("bits,g", [(2, 0), (3, 8), (4, 0)])
def test_bcd_with_block_size_one_is_the_greedy_descent(bits, g):
    X, W, H32, init = _setup(70, 120, 24, 7, bits, g)
    cd = oracle.cd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], 30, g)
    b1 = oracle.bcd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], 1, 30, seed=9, group_size=g)
    assert np.array_equal(b1["Q"], cd["Q"]) and b1["moves"].sum() == cd["committed"]


@pytest.mark.parametrize("bits,g,k", [(2, 0, 2), (3, 6, 2), (2, 0, 3)])
def test_bcd_step_is_the_best_block_move_and_loss_is_the_loss_from_x(bits, g, k):
    d_in, d_out = 12, 5
    X, W, H32, init = _setup(71, 90, d_in, d_out, bits, g)
    a = _expand(init["scale"], d_in); b = _expand(init["zero"], d_in)
    Hd = H32.astype(np.float64); Wd = W.astype(np.float64)
    seed = 21
    one = oracle.bcd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], k, 1, seed=seed, group_size=g)
    np.testing.assert_allclose(one["loss_after"], _direct_loss(X, W, init["scale"], init["zero"], one["Q"]), rtol=1e-5)
    for j in range(d_out):
        # brute force over the blocks of pi(., step 0) and all level assignments, loss from the definition
        q0 = init["Q"][:, j].astype(np.int64)
        base = (a[:, j] * q0 + b[:, j] - Wd[:, j]); base = base @ Hd @ base
        perm = oracle.bcd_perm(d_in, seed, 0)
        best, bq = base, q0
        for u in range(d_in // k):
            blk = sorted(int(x) for x in perm[k * u:k * u + k])
            for r in itertools.product(range(2 ** bits), repeat=k):
                q = q0.copy(); q[blk] = r
                e = a[:, j] * q + b[:, j] - Wd[:, j]
                l = e @ Hd @ e
                if l < best * (1 - 1e-12):
                    best, bq = l, q
        np.testing.assert_allclose(one["loss_after"][j], best, rtol=1e-9)
        assert one["moves"][j] == (0 if bq is q0 else 1)
    # many steps: the loss never rises and the moves are counted
    many = oracle.bcd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], k, 40, seed=seed, group_size=g)
    assert (many["loss_after"] <= one["loss_after"] * (1 + 1e-12)).all()
    prev = init["Q"]
    lprev = many["loss_before"]
    for T in (5, 10, 20, 40):     # prefixes of the same run (the partition depends on the step index only)
        r = oracle.bcd_solve(H32, W, bits, init["scale"], init["zero"], init["Q"], k, T, seed=seed, group_size=g)
        assert (r["loss_after"] <= lprev * (1 + 1e-12)).all()
        lprev = r["loss_after"]
    assert np.array_equal(r["Q"], many["Q"])


def test_bcd_from_the_greedy_solution_never_worse():
    X, W, H32, init = _setup(72, 200, 32, 10, 2)
    cd = oracle.cd_solve(H32, W, 2, init["scale"], init["zero"], init["Q"], 64)
    b2 = oracle.bcd_solve(H32, W, 2, init["scale"], init["zero"], cd["Q"], 2, 128, seed=1)
    _, per = oracle.layer_loss(H32, W, init["scale"], init["zero"], cd["Q"])
    np.testing.assert_allclose(b2["loss_before"], per, rtol=1e-12)
    assert (b2["loss_after"] <= b2["loss_before"]).all() and b2["moves"].sum() > 0
