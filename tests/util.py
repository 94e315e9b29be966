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
            "loss": loss, "per_col": per.cpu().numpy()}


def rel_fro(A, Bm):
    A = np.asarray(A, dtype=np.float64); Bm = np.asarray(Bm, dtype=np.float64)
    return float(np.linalg.norm(A - Bm) / np.linalg.norm(Bm))
