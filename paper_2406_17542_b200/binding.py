"""ctypes binding of the C-ABI CUDA library (``include/cdq.h``), same names as the C calls.

Argument marshalling only: every step of the path runs in the library's kernels.  torch is
used for device memory, streams and host<->device copies.  If ``libcdq.so`` has not been
built the import of any function here fails loudly; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcdq.so")
_lib = None

CDQ_OK = 0
STATUS_NAMES = {0: "CDQ_OK", 1: "CDQ_ERR_INVALID_ARG", 2: "CDQ_ERR_SHAPE", 3: "CDQ_ERR_UNSUPPORTED",
                4: "CDQ_ERR_WORKSPACE", 5: "CDQ_ERR_CUDA", 6: "CDQ_ERR_TIMEOUT"}
CDQ_F32, CDQ_BF16 = 0, 1
MODE_FAST, MODE_FP64_VERIFY = 0, 1
CALL_HESSIAN, CALL_INIT_RTN, CALL_CD_SOLVE, CALL_LAYER_LOSS, CALL_INIT_OWC_CD, CALL_BCD_SOLVE = 0, 1, 2, 3, 4, 5
CALL_CD_SOLVE_ROWS16 = 6
_MODES = {"fast": MODE_FAST, "verify": MODE_FP64_VERIFY, MODE_FAST: MODE_FAST, MODE_FP64_VERIFY: MODE_FP64_VERIFY}

EXPORTS = ["cdq_hessian", "cdq_hessian_add_lambda", "cdq_init_rtn", "cdq_init_owc_cd", "cdq_cd_solve", "cdq_cd_solve_steps", "cdq_cd_solve_with_loss", "cdq_cd_solve_rows16", "cdq_bcd_solve", "cdq_layer_loss", "cdq_layer_loss_static",
           "cdq_workspace_bytes",
           "cdq_last_device_status", "cdq_last_error_detail", "cdq_status_string", "cdq_version",
           "cdq_kernel_launches", "cdq_debug_expire_wait", "cdq_debug_set_device_status"]


class CdqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class cdq_grid_desc(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int), ("group_size", ctypes.c_int), ("n_clip", ctypes.c_int),
                ("clip_lo", ctypes.c_float), ("clip_hi", ctypes.c_float)]


class cdq_cd_stats(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_ulonglong), ("committed", ctypes.c_ulonglong),
                ("columns_converged", ctypes.c_ulonglong), ("loss_before", ctypes.c_double),
                ("loss_after", ctypes.c_double), ("kernel_ms", ctypes.c_double)]


class cdq_owc_cd_stats(ctypes.Structure):
    _fields_ = [("moves", ctypes.c_ulonglong), ("loss_before", ctypes.c_double), ("loss_after", ctypes.c_double)]


@dataclass
class Grid:
    bits: int
    group_size: int = 0
    n_clip: int = 1
    clip_lo: float = 1.0
    clip_hi: float = 1.0

    def c(self) -> cdq_grid_desc:
        return cdq_grid_desc(self.bits, self.group_size, self.n_clip, self.clip_lo, self.clip_hi)


def load():
    """Load libcdq.so and declare the signatures of include/cdq.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2406_17542_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ll, sz, ci, cf = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_size_t, ctypes.c_int, ctypes.c_float
    gp = ctypes.POINTER(cdq_grid_desc)
    lib.cdq_version.restype = ci
    lib.cdq_status_string.restype = ctypes.c_char_p
    lib.cdq_status_string.argtypes = [ci]
    lib.cdq_last_device_status.restype = ci
    lib.cdq_kernel_launches.restype = ctypes.c_ulonglong
    lib.cdq_debug_expire_wait.restype = ci
    lib.cdq_debug_expire_wait.argtypes = [ll, vp]
    lib.cdq_debug_set_device_status.restype = ci
    lib.cdq_debug_set_device_status.argtypes = [ci]
    lib.cdq_last_error_detail.restype = ctypes.c_char_p
    lib.cdq_workspace_bytes.restype = sz
    lib.cdq_workspace_bytes.argtypes = [ci, ll, ll, ll, gp, ci]
    lib.cdq_hessian.restype = ci
    lib.cdq_hessian.argtypes = [vp, ci, ll, ll, ll, cf, ci, vp, ci, vp, sz, vp]
    lib.cdq_init_rtn.restype = ci
    lib.cdq_init_rtn.argtypes = [vp, ci, ll, ll, ll, vp, gp, vp, vp, vp, vp, ci, vp, sz, vp]
    lib.cdq_init_owc_cd.restype = ci
    lib.cdq_init_owc_cd.argtypes = [vp, ci, ll, ll, ll, vp, gp, ll, vp, vp, vp, vp, ctypes.POINTER(cdq_owc_cd_stats),
                                    ci, vp, sz, vp]
    lib.cdq_cd_solve.restype = ci
    lib.cdq_cd_solve.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ci, ci, ctypes.POINTER(cdq_cd_stats), vp, sz, vp]
    lib.cdq_hessian_add_lambda.restype = ci
    lib.cdq_hessian_add_lambda.argtypes = [vp, ll, ctypes.c_float, vp]
    lib.cdq_bcd_solve.restype = ci
    lib.cdq_bcd_solve.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ci, ll, ctypes.c_ulonglong, ci,
                                  ctypes.POINTER(cdq_cd_stats), vp, sz, vp]
    lib.cdq_cd_solve_steps.restype = ci
    lib.cdq_cd_solve_steps.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ll, ci, ctypes.POINTER(cdq_cd_stats), vp, sz, vp]
    lib.cdq_cd_solve_rows16.restype = ci
    lib.cdq_cd_solve_with_loss.restype = ci
    lib.cdq_cd_solve_with_loss.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ll, ci, ctypes.POINTER(cdq_cd_stats),
                                           ctypes.POINTER(ctypes.c_double), vp, vp, sz, vp]
    lib.cdq_cd_solve_rows16.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ll, ctypes.POINTER(cdq_cd_stats), vp, sz, vp]
    lib.cdq_layer_loss.restype = ci
    lib.cdq_layer_loss.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ctypes.POINTER(ctypes.c_double), vp, ci, vp, sz, vp]
    lib.cdq_layer_loss_static.restype = ci
    lib.cdq_layer_loss_static.argtypes = [vp, vp, ci, ll, ll, ll, gp, vp, vp, vp, ctypes.POINTER(ctypes.c_double), vp, vp]
    _lib = lib
    return lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return CDQ_F32
    if t.dtype == torch.bfloat16:
        return CDQ_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != CDQ_OK:
        if status == 5:
            where += " [" + load().cdq_last_error_detail().decode() + "]"
        raise CdqError(status, where)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("device tensors required (the C ABI takes device pointers)")


class Workspace:
    """A reusable device scratch buffer handed to the library (the library never allocates)."""

    def __init__(self):
        self.buf = None

    def get(self, nbytes: int, device):
        if nbytes == 0:
            return None, 0
        if self.buf is None or self.buf.numel() < nbytes or self.buf.device != torch.device(device):
            self.buf = None
            self.buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        return self.buf.data_ptr(), self.buf.numel()


_default_ws = Workspace()


def workspace_bytes(which: int, n: int, d_in: int, d_out: int, grid: Grid | None, mode="fast") -> int:
    g = grid.c() if grid is not None else None
    return int(load().cdq_workspace_bytes(which, n, d_in, d_out, ctypes.byref(g) if g is not None else None,
                                          _MODES[mode]))


def cdq_hessian(X: torch.Tensor, lambda_rel: float = 0.0, accumulate: bool = False, out: torch.Tensor | None = None,
                mode="fast", ws: Workspace | None = None) -> torch.Tensor:
    """H = X^T X (+ lambda_rel * mean(diag) on the diagonal); X is [n, d_in] fp32 or bf16 on the device."""
    _need_cuda(X, out)
    assert X.dim() == 2 and X.stride(1) == 1
    n, d_in = X.shape
    H = out if out is not None else torch.empty((d_in, d_in), dtype=torch.float32, device=X.device)
    assert H.is_contiguous() and H.dtype == torch.float32
    ws = ws or _default_ws
    wptr, wbytes = ws.get(workspace_bytes(CALL_HESSIAN, n, d_in, 0, None, mode), X.device)
    st = load().cdq_hessian(X.data_ptr(), _dtype_code(X), n, d_in, X.stride(0), float(lambda_rel), int(accumulate),
                            H.data_ptr(), _MODES[mode], wptr, wbytes, _stream())
    _check(st, "cdq_hessian")
    return H


def cdq_hessian_add_lambda(H: torch.Tensor, lambda_rel: float) -> torch.Tensor:
    """H_ii += lambda_rel * mean(diag H), in place (for a Hessian summed from parts)."""
    _need_cuda(H)
    assert H.dim() == 2 and H.shape[0] == H.shape[1] and H.is_contiguous() and H.dtype == torch.float32
    _check(load().cdq_hessian_add_lambda(H.data_ptr(), H.shape[0], float(lambda_rel), _stream()), "cdq_hessian_add_lambda")
    return H


def cdq_init_rtn(W: torch.Tensor, grid: Grid, H: torch.Tensor | None = None, mode="fast",
                 ws: Workspace | None = None):
    """Grid + round-to-nearest codes (OWC search when grid.n_clip > 1).

    Returns (scale [d_in/g, d_out] f32, zero [d_in/g, d_out] f32, Q [d_in, d_out] u8, gamma [d_out] f32)."""
    _need_cuda(W, H)
    assert W.dim() == 2 and W.stride(1) == 1
    d_in, d_out = W.shape
    g = grid.group_size if grid.group_size > 0 else d_in
    ng = max(d_in // g, 1)
    dev = W.device
    scale = torch.empty((ng, d_out), dtype=torch.float32, device=dev)
    zero = torch.empty((ng, d_out), dtype=torch.float32, device=dev)
    Q = torch.empty((d_in, d_out), dtype=torch.uint8, device=dev)
    gamma = torch.empty((d_out,), dtype=torch.float32, device=dev)
    gd = grid.c()
    ws = ws or _default_ws
    wptr, wbytes = ws.get(workspace_bytes(CALL_INIT_RTN, 0, d_in, d_out, grid, mode), dev)
    st = load().cdq_init_rtn(W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0),
                             H.data_ptr() if H is not None else None, ctypes.byref(gd), scale.data_ptr(),
                             zero.data_ptr(), Q.data_ptr(), gamma.data_ptr(), _MODES[mode], wptr, wbytes, _stream())
    _check(st, "cdq_init_rtn")
    return scale, zero, Q, gamma


def cdq_init_owc_cd(W: torch.Tensor, grid: Grid, H: torch.Tensor, steps: int = 0, mode="fast",
                    ws: Workspace | None = None):
    """OWC-CD (Algorithm 3): one clipping strength per group, chosen by greedy descent over the groups.

    Returns (scale, zero, Q, gamma [d_in/g, d_out] f32, stats dict)."""
    _need_cuda(W, H)
    assert W.dim() == 2 and W.stride(1) == 1 and H.is_contiguous() and H.dtype == torch.float32
    d_in, d_out = W.shape
    g = grid.group_size if grid.group_size > 0 else d_in
    ng = max(d_in // g, 1)
    dev = W.device
    scale = torch.empty((ng, d_out), dtype=torch.float32, device=dev)
    zero = torch.empty((ng, d_out), dtype=torch.float32, device=dev)
    Q = torch.empty((d_in, d_out), dtype=torch.uint8, device=dev)
    gamma = torch.empty((ng, d_out), dtype=torch.float32, device=dev)
    gd = grid.c()
    stats = cdq_owc_cd_stats()
    ws = ws or _default_ws
    wptr, wbytes = ws.get(workspace_bytes(CALL_INIT_OWC_CD, 0, d_in, d_out, grid, mode), dev)
    st = load().cdq_init_owc_cd(W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0), H.data_ptr(), ctypes.byref(gd),
                                int(steps), scale.data_ptr(), zero.data_ptr(), Q.data_ptr(), gamma.data_ptr(),
                                ctypes.byref(stats), _MODES[mode], wptr, wbytes, _stream())
    _check(st, "cdq_init_owc_cd")
    return scale, zero, Q, gamma, {"moves": stats.moves, "loss_before": stats.loss_before,
                                   "loss_after": stats.loss_after}


def cdq_cd_solve(H: torch.Tensor, W: torch.Tensor, grid: Grid, scale: torch.Tensor, zero: torch.Tensor,
                 Q: torch.Tensor, passes: int, mode="fast", want_stats: bool = True, ws: Workspace | None = None,
                 steps_per_col: int | None = None, rows16: bool = False):
    """Greedy coordinate descent on every column; Q is updated in place.  Returns the stats dict (or None).
    With steps_per_col the budget is that many steps per column (cdq_cd_solve_steps) instead of passes * d_in.
    rows16: the update reads its rows from a bf16 copy of H (cdq_cd_solve_rows16)."""
    _need_cuda(H, W, scale, zero, Q)
    d_in, d_out = W.shape
    assert H.shape == (d_in, d_in) and H.is_contiguous() and H.dtype == torch.float32
    assert Q.shape == (d_in, d_out) and Q.is_contiguous() and Q.dtype == torch.uint8
    assert scale.is_contiguous() and zero.is_contiguous() and W.stride(1) == 1
    gd = grid.c()
    stats = cdq_cd_stats()
    ws = ws or _default_ws
    if rows16:
        wptr, wbytes = ws.get(workspace_bytes(CALL_CD_SOLVE_ROWS16, 0, d_in, d_out, grid, mode), W.device)
        st = load().cdq_cd_solve_rows16(H.data_ptr(), W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0), ctypes.byref(gd),
                                        scale.data_ptr(), zero.data_ptr(), Q.data_ptr(),
                                        int(passes * d_in if steps_per_col is None else steps_per_col),
                                        ctypes.byref(stats) if want_stats else None, wptr, wbytes, _stream())
        _check(st, "cdq_cd_solve_rows16")
        if not want_stats:
            return None
        return {"steps": stats.steps, "committed": stats.committed, "columns_converged": stats.columns_converged,
                "loss_before": stats.loss_before, "loss_after": stats.loss_after, "kernel_ms": stats.kernel_ms}
    wptr, wbytes = ws.get(workspace_bytes(CALL_CD_SOLVE, 0, d_in, d_out, grid, mode), W.device)
    fn = load().cdq_cd_solve if steps_per_col is None else load().cdq_cd_solve_steps
    st = fn(H.data_ptr(), W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0), ctypes.byref(gd),
            scale.data_ptr(), zero.data_ptr(), Q.data_ptr(), int(passes if steps_per_col is None else steps_per_col),
            _MODES[mode], ctypes.byref(stats) if want_stats else None, wptr, wbytes, _stream())
    _check(st, "cdq_cd_solve")
    if not want_stats:
        return None
    return {"steps": stats.steps, "committed": stats.committed, "columns_converged": stats.columns_converged,
            "loss_before": stats.loss_before, "loss_after": stats.loss_after, "kernel_ms": stats.kernel_ms}


def cdq_cd_solve_with_loss(H: torch.Tensor, W: torch.Tensor, grid: Grid, scale: torch.Tensor, zero: torch.Tensor,
                           Q: torch.Tensor, steps_per_col: int, mode="fast", per_col: bool | torch.Tensor = False,
                           ws: Workspace | None = None):
    """Greedy coordinate descent (Q updated in place) and the loss of its result from the descent's own
    gradient.  Returns (stats, loss) or (stats, loss, per_col)."""
    _need_cuda(H, W, scale, zero, Q)
    d_in, d_out = W.shape
    assert H.shape == (d_in, d_in) and H.is_contiguous() and H.dtype == torch.float32
    assert Q.shape == (d_in, d_out) and Q.is_contiguous() and Q.dtype == torch.uint8
    assert scale.is_contiguous() and zero.is_contiguous() and W.stride(1) == 1
    gd = grid.c()
    stats = cdq_cd_stats()
    loss = ctypes.c_double(0.0)
    cols = None
    if isinstance(per_col, torch.Tensor):
        cols = per_col
        assert cols.is_cuda and cols.dtype == torch.float64 and cols.is_contiguous() and cols.numel() == d_out
    elif per_col:
        cols = torch.empty(d_out, dtype=torch.float64, device=W.device)
    ws = ws or _default_ws
    wptr, wbytes = ws.get(workspace_bytes(CALL_CD_SOLVE, 0, d_in, d_out, grid, mode), W.device)
    st = load().cdq_cd_solve_with_loss(H.data_ptr(), W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0), ctypes.byref(gd),
                                       scale.data_ptr(), zero.data_ptr(), Q.data_ptr(), int(steps_per_col), _MODES[mode],
                                       ctypes.byref(stats), ctypes.byref(loss), cols.data_ptr() if cols is not None else None,
                                       wptr, wbytes, _stream())
    _check(st, "cdq_cd_solve_with_loss")
    sd = {"steps": stats.steps, "committed": stats.committed, "columns_converged": stats.columns_converged,
          "loss_before": stats.loss_before, "loss_after": stats.loss_after, "kernel_ms": stats.kernel_ms}
    return (sd, loss.value, cols) if cols is not None else (sd, loss.value)


def cdq_bcd_solve(H: torch.Tensor, W: torch.Tensor, grid: Grid, scale: torch.Tensor, zero: torch.Tensor,
                  Q: torch.Tensor, block: int, steps_per_col: int, seed: int = 0, mode="fast",
                  want_stats: bool = True, ws: Workspace | None = None):
    """Block coordinate descent with random blocks of `block` coordinates; Q is updated in place."""
    _need_cuda(H, W, scale, zero, Q)
    d_in, d_out = W.shape
    assert H.shape == (d_in, d_in) and H.is_contiguous() and H.dtype == torch.float32
    assert Q.shape == (d_in, d_out) and Q.is_contiguous() and Q.dtype == torch.uint8
    assert scale.is_contiguous() and zero.is_contiguous() and W.stride(1) == 1
    gd = grid.c()
    stats = cdq_cd_stats()
    ws = ws or _default_ws
    wptr, wbytes = ws.get(workspace_bytes(CALL_BCD_SOLVE, int(steps_per_col), d_in, d_out, grid, mode), W.device)
    st = load().cdq_bcd_solve(H.data_ptr(), W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0), ctypes.byref(gd),
                              scale.data_ptr(), zero.data_ptr(), Q.data_ptr(), int(block), int(steps_per_col),
                              int(seed) & 0xFFFFFFFFFFFFFFFF, _MODES[mode], ctypes.byref(stats) if want_stats else None,
                              wptr, wbytes, _stream())
    _check(st, "cdq_bcd_solve")
    if not want_stats:
        return None
    return {"steps": stats.steps, "committed": stats.committed, "columns_converged": stats.columns_converged,
            "loss_before": stats.loss_before, "loss_after": stats.loss_after, "kernel_ms": stats.kernel_ms}


def cdq_layer_loss(H: torch.Tensor, W: torch.Tensor, grid: Grid, scale: torch.Tensor, zero: torch.Tensor,
                   Q: torch.Tensor, per_col: bool = False, mode="fast", ws: Workspace | None = None):
    """sum_j e_j^T H e_j.  Returns the total (python float), or (total, per-column fp64 tensor)."""
    _need_cuda(H, W, scale, zero, Q)
    d_in, d_out = W.shape
    gd = grid.c()
    loss = ctypes.c_double(0.0)
    pc = torch.empty((d_out,), dtype=torch.float64, device=W.device) if per_col else None
    ws = ws or _default_ws
    wptr, wbytes = ws.get(workspace_bytes(CALL_LAYER_LOSS, 0, d_in, d_out, grid, mode), W.device)
    st = load().cdq_layer_loss(H.data_ptr(), W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0), ctypes.byref(gd),
                               scale.data_ptr(), zero.data_ptr(), Q.data_ptr(), ctypes.byref(loss),
                               pc.data_ptr() if pc is not None else None, _MODES[mode], wptr, wbytes, _stream())
    _check(st, "cdq_layer_loss")
    return (loss.value, pc) if per_col else loss.value


STATIC_SCRATCH_BYTES = 20 * 1024 * 1024


def cdq_layer_loss_static(H: torch.Tensor, W: torch.Tensor, grid: Grid, scale: torch.Tensor, zero: torch.Tensor,
                          Q: torch.Tensor, per_col: torch.Tensor | None = None) -> float:
    """The layer loss without a workspace: for callers that may not allocate device memory (a
    frozen memory pool, a latency-critical path).  Scratch is a fixed STATIC_SCRATCH_BYTES
    array inside the library, shared by all calls on a GPU, so calls must not overlap; layers
    whose residual does not fit are refused with CDQ_ERR_WORKSPACE.  `per_col` (fp64 [d_out]
    on the device), if given, receives the per-column losses -- this binding allocates nothing
    either.  The first call on a device should happen during set-up."""
    d_in, d_out = W.shape
    gd = grid.c()
    loss = ctypes.c_double(0.0)
    st = load().cdq_layer_loss_static(H.data_ptr(), W.data_ptr(), _dtype_code(W), d_in, d_out, W.stride(0),
                                      ctypes.byref(gd), scale.data_ptr(), zero.data_ptr(), Q.data_ptr(),
                                      ctypes.byref(loss), per_col.data_ptr() if per_col is not None else None,
                                      _stream())
    if status_is_workspace(st):
        raise CdqError(st, "cdq_layer_loss_static [" + load().cdq_last_error_detail().decode() + "]")
    _check(st, "cdq_layer_loss_static")
    return loss.value


def status_is_workspace(st: int) -> bool:
    return st == 4


def quantize_layer(X: torch.Tensor, W: torch.Tensor, grid: Grid, passes: int, lambda_rel: float = 0.0, mode="fast",
                   device="cuda:0", ws: Workspace | None = None, return_host: bool | None = None,
                   init: str = "rtn", steps_per_col: int | None = None, bcd_steps: int = 0, seed: int = 0) -> dict:
    """The whole hot path for one layer: Hessian, grid/codes, greedy CD, loss.

    X and W may live on the host (pinned memory makes the copies asynchronous): they are then
    copied to `device` first and the codes, scales and zeros are copied back, so that a caller
    holding host buffers gets host results.  All compute is the library's calls.

    The paper's variants around the main loop: init="owc_cd" takes the grid from cdq_init_owc_cd
    (per-group clipping strengths, needs grid.n_clip > 1) instead of cdq_init_rtn; steps_per_col
    gives the descent's budget in steps per column instead of passes * d_in; bcd_steps > 0 runs
    that many steps of block coordinate descent with random pairs from the greedy solution."""
    if init not in ("rtn", "owc_cd"):
        raise ValueError("init must be 'rtn' or 'owc_cd'")
    on_host = not X.is_cuda
    if return_host is None:
        return_host = on_host
    Xd = X.to(device, non_blocking=True) if not X.is_cuda else X
    Wd = W.to(device, non_blocking=True) if not W.is_cuda else W
    H = cdq_hessian(Xd, lambda_rel=lambda_rel, mode=mode, ws=ws)
    if init == "owc_cd":
        scale, zero, Q, gamma, _ = cdq_init_owc_cd(Wd, grid, H, mode=mode, ws=ws)
    else:
        scale, zero, Q, gamma = cdq_init_rtn(Wd, grid, H=H if grid.n_clip > 1 else None, mode=mode, ws=ws)
    budget = passes * Wd.shape[0] if steps_per_col is None else steps_per_col
    if bcd_steps > 0:
        stats = cdq_cd_solve(H, Wd, grid, scale, zero, Q, passes, mode=mode, ws=ws, steps_per_col=steps_per_col)
        out = {"H": H, "scale": scale, "zero": zero, "Q": Q, "gamma": gamma, "stats": stats}
        out["bcd_stats"] = cdq_bcd_solve(H, Wd, grid, scale, zero, Q, 2, bcd_steps, seed=seed, mode=mode, ws=ws)
        out["loss"] = cdq_layer_loss(H, Wd, grid, scale, zero, Q, mode=mode, ws=ws)
    else:   # the descent hands back the loss of its result
        stats, loss = cdq_cd_solve_with_loss(H, Wd, grid, scale, zero, Q, budget, mode=mode, ws=ws)
        out = {"H": H, "scale": scale, "zero": zero, "Q": Q, "gamma": gamma, "stats": stats, "loss": loss}
    if return_host:
        for k in ("scale", "zero", "Q"):
            out[k] = out[k].to("cpu", non_blocking=False)
    return out


_copy_streams: dict = {}


def quantize_layers(layers, grid: Grid, passes: int, device="cuda:0", ws: Workspace | None = None,
                    host_buffers: dict | None = None, **kw):
    """Generator over an iterable of (X, W) pairs held in (pinned) host memory: yields quantize_layer's result for
    every layer in turn, with codes, scales and zeros back in pinned host buffers.

    The inputs of layer k + 1 are uploaded on a second stream while layer k computes (two input buffers on the
    device), so that from the second layer on the host-to-device copy costs nothing unless it is longer than
    the layer's compute.  The host buffers of a result are reused by the next layer of the same shape: copy what
    must outlive the next iteration (host_buffers: a dict that keeps them across calls).  Keyword arguments are
    quantize_layer's (lambda_rel, mode, init, ...)."""
    dev = torch.device(device)
    if dev not in _copy_streams:
        _copy_streams[dev] = torch.cuda.Stream(dev)
    copy_stream = _copy_streams[dev]
    main = torch.cuda.current_stream(dev)
    host_out: dict = host_buffers if host_buffers is not None else {}
    it = iter(layers)

    def upload(pair):
        X, W = pair
        with torch.cuda.stream(copy_stream):
            Xd = X.to(dev, non_blocking=True)
            Wd = W.to(dev, non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(copy_stream)
        return Xd, Wd, ev

    nxt = next(it, None)
    pending = upload(nxt) if nxt is not None else None
    while pending is not None:
        Xd, Wd, ev = pending
        nxt = next(it, None)
        pending = upload(nxt) if nxt is not None else None   # in flight while this layer computes
        main.wait_event(ev)
        out = quantize_layer(Xd, Wd, grid, passes, device=device, ws=ws, return_host=False, **kw)
        Xd.record_stream(main)
        Wd.record_stream(main)
        for k in ("scale", "zero", "Q"):
            t = out[k]
            key = (k, tuple(t.shape), t.dtype)
            if key not in host_out:
                host_out[key] = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
            host_out[key].copy_(t, non_blocking=True)
            out[k] = host_out[key]
        main.synchronize()
        yield out
