"""Seeded synthetic layers shaped like the paper's Gemma / PaLM2 workloads.

This module only draws random inputs (calibration activations X and weights W)
and names the five benchmark configurations.  It holds none of the method's
arithmetic, so both the CUDA library's callers and the CPU oracle's callers may
use it: the same buffers are handed to both sides.

Recipe (stand-in for real calibration activations and model weights, which are
not available offline): per-feature scales s_f = exp(sigma * N(0,1)); a random
fraction of "outlier" features is multiplied by 20; entries are N(0,1) or
Student-t(nu=4) drawn as N / sqrt(chi2_4 / 4); X = entries * s_f rounded to the
storage type; W ~ N(0, sigma_w) rounded to its storage type.  Everything comes
from one torch.Generator seeded per configuration, drawn in row chunks so that
the largest layers never need more than the result plus one chunk.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    d_in: int
    d_out: int
    n: int                 # calibration rows
    x_dtype: str           # "f32" | "bf16"
    w_dtype: str           # "f32" | "bf16"
    feat_sigma: float      # sigma of the log-normal per-feature scale
    outlier_frac: float    # fraction of features multiplied by 20
    student_t: bool        # Student-t(nu=4) entries instead of N(0,1)
    w_sigma: float
    bits: int
    group_size: int        # 0 => per-channel
    n_clip: int            # <=1 => MinMax
    clip_lo: float
    clip_hi: float
    passes: int
    seed: int

    def scaled(self, **kw) -> "LayerConfig":
        """A smaller (or otherwise altered) copy, e.g. for tests."""
        return replace(self, **kw)


CONFIGS = {
    "C0": LayerConfig("C0", 256, 256, 1024, "f32", "f32", 1.0, 0.0, False, 0.02, 4, 0, 1, 1.0, 1.0, 1, 0),
    "C1": LayerConfig("C1", 2048, 16384, 65536, "bf16", "bf16", 1.5, 0.01, False, 0.02, 3, 0, 1, 1.0, 1.0, 2, 1),
    "C2": LayerConfig("C2", 4096, 4096, 131072, "bf16", "f32", 1.5, 0.01, False, 0.015, 2, 128, 20, 0.5, 1.0, 3, 2),
    "C3": LayerConfig("C3", 14336, 4096, 131072, "bf16", "f32", 1.0, 0.0, True, 0.01, 4, 0, 1, 1.0, 1.0, 2, 3),
    "C4": LayerConfig("C4", 18432, 73728, 262144, "bf16", "f32", 1.5, 0.0, True, 0.008, 3, 128, 20, 0.5, 1.0, 1, 4),
}

_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


def torch_dtype(name: str) -> torch.dtype:
    return _TORCH_DTYPE[name]


def make_generator(cfg: LayerConfig, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(1000003 * cfg.seed + 12345)
    return g


def feature_scales(cfg: LayerConfig, gen: torch.Generator, device="cpu") -> torch.Tensor:
    s = torch.exp(cfg.feat_sigma * torch.randn(cfg.d_in, generator=gen, device=device))
    if cfg.outlier_frac > 0:
        k = max(1, int(round(cfg.outlier_frac * cfg.d_in)))
        idx = torch.randperm(cfg.d_in, generator=gen, device=device)[:k]
        s[idx] *= 20.0
    return s


def make_x(cfg: LayerConfig, device="cpu", chunk_rows: int = 8192) -> torch.Tensor:
    """Calibration inputs X [n, d_in] in the configuration's storage type."""
    gen = make_generator(cfg, device)
    s = feature_scales(cfg, gen, device)
    X = torch.empty((cfg.n, cfg.d_in), dtype=torch_dtype(cfg.x_dtype), device=device)
    for r0 in range(0, cfg.n, chunk_rows):
        r1 = min(cfg.n, r0 + chunk_rows)
        z = torch.randn((r1 - r0, cfg.d_in), generator=gen, device=device)
        if cfg.student_t:
            chi = torch.zeros_like(z)
            for _ in range(4):
                chi += torch.randn((r1 - r0, cfg.d_in), generator=gen, device=device) ** 2
            z = z / torch.sqrt(chi / 4.0)
        X[r0:r1] = (z * s).to(X.dtype)
    return X


def make_w(cfg: LayerConfig, device="cpu", chunk_rows: int = 2048) -> torch.Tensor:
    """Weights W [d_in, d_out] in the configuration's storage type."""
    gen = torch.Generator(device=device)
    gen.manual_seed(7919 * cfg.seed + 777)
    W = torch.empty((cfg.d_in, cfg.d_out), dtype=torch_dtype(cfg.w_dtype), device=device)
    for r0 in range(0, cfg.d_in, chunk_rows):
        r1 = min(cfg.d_in, r0 + chunk_rows)
        W[r0:r1] = (cfg.w_sigma * torch.randn((r1 - r0, cfg.d_out), generator=gen, device=device)).to(W.dtype)
    return W


def make_layer(cfg: LayerConfig, device="cpu"):
    """(X, W) for one configuration."""
    return make_x(cfg, device), make_w(cfg, device)
