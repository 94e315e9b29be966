"""Python face of the fp64 CPU oracle (TEST INFRASTRUCTURE, not product code).

Loads ``cdq_oracle.c`` (compiled on first use with gcc, OpenMP, no FMA
contraction) through ctypes.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library never
does, and nothing here imports the CUDA binding.

Every function takes the layer in the paper's orientation (Section 3,
Notation): X is [n, d_in], W is [d_in, d_out]; codes Q are [d_in, d_out] u8;
scale a and zero b are [d_in/g, d_out] fp32 (one row when per-channel).
Inputs may be numpy arrays or CPU torch tensors of any float type; they are
widened exactly to fp64 before the C code sees them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cdq_oracle.c")
_LIB = os.path.join(_HERE, "libcdq_oracle.so")
_lock = threading.Lock()
_lib = None

_i64 = ctypes.c_longlong
_dp = ctypes.POINTER(ctypes.c_double)
_fp = ctypes.POINTER(ctypes.c_float)
_u8p = ctypes.POINTER(ctypes.c_ubyte)
_ip = ctypes.POINTER(ctypes.c_int)
_i64p = ctypes.POINTER(ctypes.c_longlong)
_u64p = ctypes.POINTER(ctypes.c_ulonglong)


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared object next to it."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared",
                   "-fPIC", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    lib.cdqo_num_threads.restype = ctypes.c_int
    lib.cdqo_gamma.restype = ctypes.c_double
    lib.cdqo_gamma.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_double]
    lib.cdqo_hessian.argtypes = [_dp, _i64, _i64, ctypes.c_double, _dp, _fp]
    lib.cdqo_hessian_entries.argtypes = [_dp, _i64, _i64, _i64p, _i64p, _i64, _dp]
    lib.cdqo_bcd_perm.restype = _i64
    lib.cdqo_bcd_perm.argtypes = [_i64, _i64, ctypes.c_ulonglong, _i64]
    lib.cdqo_bcd_solve.argtypes = [_fp, _dp, _i64, _i64, ctypes.c_int, _i64, _fp, _fp, _u8p, ctypes.c_int, _i64,
                                   ctypes.c_ulonglong, _i64p, _dp, _dp]
    lib.cdqo_owc_cd.argtypes = [_dp, _i64, _i64, _fp, ctypes.c_int, _i64, ctypes.c_int, ctypes.c_double,
                                ctypes.c_double, _i64, _fp, _fp, _u8p, _ip, _i64p, _dp, _dp]
    lib.cdqo_init_rtn.argtypes = [_dp, _i64, _i64, _fp, ctypes.c_int, _i64, ctypes.c_int,
                                  ctypes.c_double, ctypes.c_double, _fp, _fp, _u8p, _ip, _dp]
    lib.cdqo_gradient.argtypes = [_fp, _dp, _i64, _i64, _i64, _fp, _fp, _u8p, _dp]
    lib.cdqo_cd_solve.argtypes = [_fp, _dp, _i64, _i64, ctypes.c_int, _i64, _fp, _fp, _u8p, _i64,
                                  _u64p, _dp, _i64, _ip, _ip, _dp, _i64p, _dp]
    lib.cdqo_cd_code_units.restype = _i64
    lib.cdqo_cd_code_units.argtypes = [_fp, _dp, _dp, _dp, _i64, ctypes.c_int, _u8p, _i64, _ip, _ip]
    lib.cdqo_layer_loss.argtypes = [_fp, _dp, _i64, _i64, _i64, _fp, _fp, _u8p, _dp, _dp]
    _lib = lib
    return lib


def _f64(x) -> np.ndarray:
    """Widen any float array (numpy, or torch incl. bf16) exactly to contiguous fp64."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _f32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    x = np.asarray(x)
    assert x.dtype == np.float32, "expected an fp32 array"
    return np.ascontiguousarray(x)


def _u8(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    x = np.asarray(x)
    assert x.dtype == np.uint8
    return np.ascontiguousarray(x)


def _ptr(a, t):
    return a.ctypes.data_as(t) if a is not None else None


def num_threads() -> int:
    return int(_load().cdqo_num_threads())


def gamma_grid(n_clip: int, lo: float, hi: float) -> np.ndarray:
    """Clipping grid Gamma: n_clip points from lo to hi inclusive (one point => gamma = 1)."""
    lib = _load()
    n = max(int(n_clip), 1)
    return np.array([lib.cdqo_gamma(k, n, float(lo), float(hi)) for k in range(n)])


def hessian(X, lambda_rel: float = 0.0):
    """H = X^T X (Section 3, Notation).  Returns (H fp64, H rounded to fp32)."""
    X = _f64(X)
    n, d_in = X.shape
    H64 = np.empty((d_in, d_in), dtype=np.float64)
    H32 = np.empty((d_in, d_in), dtype=np.float32)
    rc = _load().cdqo_hessian(_ptr(X, _dp), n, d_in, float(lambda_rel), _ptr(H64, _dp), _ptr(H32, _fp))
    assert rc == 0, rc
    return H64, H32


def hessian_entries(X, rows, cols) -> np.ndarray:
    """Selected entries H[rows[s], cols[s]] of X^T X in fp64."""
    X = _f64(X)
    n, d_in = X.shape
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    out = np.empty(rows.shape[0], dtype=np.float64)
    rc = _load().cdqo_hessian_entries(_ptr(X, _dp), n, d_in, _ptr(rows, _i64p), _ptr(cols, _i64p),
                                      rows.shape[0], _ptr(out, _dp))
    assert rc == 0, rc
    return out


def init_rtn(W, bits: int, group_size: int = 0, n_clip: int = 1, clip_lo: float = 1.0,
             clip_hi: float = 1.0, H=None, want_loss_table: bool = False) -> dict:
    """MinMax / OWC grid and round-to-nearest codes (Eq. 2 and the gamma search after it)."""
    W = _f64(W)
    d_in, d_out = W.shape
    g = group_size if group_size > 0 else d_in
    ng = d_in // g
    Hf = _f32(H) if H is not None else None
    scale = np.empty((ng, d_out), dtype=np.float32)
    zero = np.empty((ng, d_out), dtype=np.float32)
    Q = np.empty((d_in, d_out), dtype=np.uint8)
    gidx = np.zeros(d_out, dtype=np.int32)
    nk = max(int(n_clip), 1)
    table = np.zeros((nk, d_out), dtype=np.float64) if (want_loss_table and nk > 1) else None
    rc = _load().cdqo_init_rtn(_ptr(W, _dp), d_in, d_out, _ptr(Hf, _fp), int(bits), int(group_size),
                               int(n_clip), float(clip_lo), float(clip_hi), _ptr(scale, _fp),
                               _ptr(zero, _fp), _ptr(Q, _u8p), _ptr(gidx, _ip), _ptr(table, _dp))
    assert rc == 0, rc
    return {"scale": scale, "zero": zero, "Q": Q, "gamma_idx": gidx,
            "gamma": gamma_grid(n_clip, clip_lo, clip_hi)[gidx], "loss_table": table}


def owc_cd(H, W, bits: int, group_size: int, n_clip: int, clip_lo: float, clip_hi: float, steps: int) -> dict:
    """OWC-CD (Algorithm 3): greedy descent over the clipping strengths of a column's groups,
    every group starting at the last grid point; `steps` changes per column at most."""
    Hf, W = _f32(H), _f64(W)
    d_in, d_out = W.shape
    g = group_size if group_size > 0 else d_in
    ng = d_in // g
    scale = np.empty((ng, d_out), dtype=np.float32)
    zero = np.empty((ng, d_out), dtype=np.float32)
    Q = np.empty((d_in, d_out), dtype=np.uint8)
    gidx = np.zeros((ng, d_out), dtype=np.int32)
    moves = np.zeros(d_out, dtype=np.int64)
    lb = np.zeros(d_out, dtype=np.float64)
    la = np.zeros(d_out, dtype=np.float64)
    rc = _load().cdqo_owc_cd(_ptr(W, _dp), d_in, d_out, _ptr(Hf, _fp), int(bits), int(group_size), int(n_clip),
                             float(clip_lo), float(clip_hi), int(steps), _ptr(scale, _fp), _ptr(zero, _fp),
                             _ptr(Q, _u8p), _ptr(gidx, _ip), _ptr(moves, _i64p), _ptr(lb, _dp), _ptr(la, _dp))
    assert rc == 0, rc
    return {"scale": scale, "zero": zero, "Q": Q, "gamma_idx": gidx, "moves": moves,
            "loss_before": lb, "loss_after": la}


def bcd_perm(d_in: int, seed: int, step: int) -> np.ndarray:
    """The pseudo-random permutation pi that cuts the coordinates into blocks at one step (the same for every column)."""
    lib = _load()
    return np.array([lib.cdqo_bcd_perm(x, d_in, seed, step) for x in range(d_in)], dtype=np.int64)


def bcd_solve(H, W, bits: int, scale, zero, Q, k: int, steps_per_col: int, seed: int = 0, group_size: int = 0) -> dict:
    """Block coordinate descent with random blocks of size k (Algorithm 2 / Algorithm 5), from the codes Q."""
    Hf, W, scale, zero = _f32(H), _f64(W), _f32(scale), _f32(zero)
    Q = np.array(_u8(Q), copy=True)
    d_in, d_out = W.shape
    moves = np.zeros(d_out, dtype=np.int64)
    lb = np.zeros(d_out, dtype=np.float64)
    la = np.zeros(d_out, dtype=np.float64)
    rc = _load().cdqo_bcd_solve(_ptr(Hf, _fp), _ptr(W, _dp), d_in, d_out, int(bits), int(group_size), _ptr(scale, _fp),
                                _ptr(zero, _fp), _ptr(Q, _u8p), int(k), int(steps_per_col), int(seed),
                                _ptr(moves, _i64p), _ptr(lb, _dp), _ptr(la, _dp))
    assert rc == 0, rc
    return {"Q": Q, "moves": moves, "loss_before": lb, "loss_after": la}


def gradient(H, W, scale, zero, Q, group_size: int = 0) -> np.ndarray:
    """G = 2 H (W_hat - W), returned as [d_out, d_in] fp64 (the gradient step of Algorithm 1, weight units)."""
    Hf, W, scale, zero, Q = _f32(H), _f64(W), _f32(scale), _f32(zero), _u8(Q)
    d_in, d_out = W.shape
    G = np.empty((d_out, d_in), dtype=np.float64)
    rc = _load().cdqo_gradient(_ptr(Hf, _fp), _ptr(W, _dp), d_in, d_out, int(group_size),
                               _ptr(scale, _fp), _ptr(zero, _fp), _ptr(Q, _u8p), _ptr(G, _dp))
    assert rc == 0, rc
    return G


def cd_solve(H, W, bits: int, scale, zero, Q, steps_per_col: int, group_size: int = 0,
             trace_col: int = -1, want_G: bool = False) -> dict:
    """Greedy coordinate descent (the loop of Algorithm 1 / Algorithm 4) on every column.

    Returns the new codes (the input Q is not modified) and the statistics."""
    Hf, W, scale, zero = _f32(H), _f64(W), _f32(scale), _f32(zero)
    Q = _u8(Q).copy()
    d_in, d_out = W.shape
    T = int(steps_per_col)
    stats = np.zeros(3, dtype=np.uint64)
    loss = np.zeros(2, dtype=np.float64)
    moves = np.zeros(d_out, dtype=np.int64)
    ti = tr = td = None
    if trace_col >= 0:
        ti = np.full(max(T, 1), -1, dtype=np.int32)
        tr = np.full(max(T, 1), -1, dtype=np.int32)
        td = np.zeros(max(T, 1), dtype=np.float64)
    G = np.empty((d_out, d_in), dtype=np.float64) if want_G else None
    rc = _load().cdqo_cd_solve(_ptr(Hf, _fp), _ptr(W, _dp), d_in, d_out, int(bits), int(group_size),
                               _ptr(scale, _fp), _ptr(zero, _fp), _ptr(Q, _u8p), T,
                               _ptr(stats, _u64p), _ptr(loss, _dp), int(trace_col), _ptr(ti, _ip),
                               _ptr(tr, _ip), _ptr(td, _dp), _ptr(moves, _i64p), _ptr(G, _dp))
    assert rc == 0, rc
    out = {"Q": Q, "steps": int(stats[0]), "committed": int(stats[1]),
           "columns_converged": int(stats[2]), "loss_before": float(loss[0]),
           "loss_after": float(loss[1]), "moves_per_col": moves, "G": G}
    if trace_col >= 0:
        m = int(moves[trace_col])
        out["trace"] = {"i": ti[:m].copy(), "r": tr[:m].copy(), "delta": td[:m].copy()}
    return out


def cd_code_units(H, w, a_full, b_full, bits: int, q0, steps: int) -> dict:
    """Literal code-unit iteration of Algorithm 4 (Algorithm 1 for a constant scale), one column."""
    Hf, w, a_full, b_full = _f32(H), _f64(w), _f64(a_full), _f64(b_full)
    q = _u8(q0).copy()
    d_in = w.shape[0]
    T = int(steps)
    ti = np.full(max(T, 1), -1, dtype=np.int32)
    tr = np.full(max(T, 1), -1, dtype=np.int32)
    m = _load().cdqo_cd_code_units(_ptr(Hf, _fp), _ptr(w, _dp), _ptr(a_full, _dp), _ptr(b_full, _dp),
                                   d_in, int(bits), _ptr(q, _u8p), T, _ptr(ti, _ip), _ptr(tr, _ip))
    return {"q": q, "moves": int(m), "trace_i": ti[:m].copy(), "trace_r": tr[:m].copy()}


def layer_loss(H, W, scale, zero, Q, group_size: int = 0):
    """sum_j e_j^T H e_j with e = W_hat - W (Eq. 1 with H = X^T X).  Returns (total, per column)."""
    Hf, W, scale, zero, Q = _f32(H), _f64(W), _f32(scale), _f32(zero), _u8(Q)
    d_in, d_out = W.shape
    per = np.empty(d_out, dtype=np.float64)
    tot = ctypes.c_double(0.0)
    rc = _load().cdqo_layer_loss(_ptr(Hf, _fp), _ptr(W, _dp), d_in, d_out, int(group_size),
                                 _ptr(scale, _fp), _ptr(zero, _fp), _ptr(Q, _u8p), _ptr(per, _dp),
                                 ctypes.byref(tot))
    assert rc == 0, rc
    return float(tot.value), per
