"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the method: it only draws operands.  Both
the CUDA path's tests and the CPU oracle's tests take their inputs from here.

Recipes (all fp32):
  * activations  X ~ N(0, 1)
  * weights      W ~ N(0, 0.05^2)
  * gradients    G ~ 1e-3 * Student-t(nu=3)         (heavy-tailed)
  * sweep operands: Student-t(nu=3) with 0.1 % of the entries scaled by 50
"""
from __future__ import annotations

import numpy as np


def activations(rows: int, cols: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng([seed, 1])
    return rng.standard_normal((rows, cols), dtype=np.float32)


def weights(rows: int, cols: int, seed: int, std: float = 0.05) -> np.ndarray:
    rng = np.random.default_rng([seed, 2])
    return (rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)).astype(np.float32)


def gradients(rows: int, cols: int, seed: int, scale: float = 1e-3) -> np.ndarray:
    rng = np.random.default_rng([seed, 3])
    return (rng.standard_t(3.0, size=(rows, cols)) * scale).astype(np.float32)


def heavy_tailed(rows: int, cols: int, seed: int, outlier_frac: float = 1e-3,
                 outlier_scale: float = 50.0) -> np.ndarray:
    """Student-t(3) with a Bernoulli(outlier_frac) mask of entries scaled up."""
    rng = np.random.default_rng([seed, 4])
    x = rng.standard_t(3.0, size=(rows, cols)).astype(np.float32)
    mask = rng.random((rows, cols)) < outlier_frac
    x[mask] *= np.float32(outlier_scale)
    return x


def heavy_tailed_torch(rows: int, cols: int, seed: int, device, outlier_frac: float = 1e-3,
                       outlier_scale: float = 50.0, chunk_rows: int = 2048):
    """Same distribution as `heavy_tailed`, drawn with a seeded torch generator
    on `device` (used for operands too large to draw on the host).  Student-t(3)
    = N(0,1) / sqrt(chi2_3 / 3)."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    out = torch.empty((rows, cols), dtype=torch.float32, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        shp = (r1 - r0, cols)
        z = torch.randn(shp, generator=gen, device=device)
        chi = torch.zeros(shp, device=device)
        for _ in range(3):
            chi += torch.randn(shp, generator=gen, device=device) ** 2
        t = z / torch.sqrt(chi / 3.0)
        mask = torch.rand(shp, generator=gen, device=device) < outlier_frac
        t = torch.where(mask, t * outlier_scale, t)
        out[r0:r1] = t
    return out


def single_layer(seed: int = 0, Nb: int = 32, D: int = 128, C: int = 64):
    """One linear layer: X[Nb,D], W[D,C], G[Nb,C]."""
    return activations(Nb, D, seed), weights(D, C, seed), gradients(Nb, C, seed)
