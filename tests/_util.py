"""Helpers shared by the parity tests: error metric, tolerances, GPU state <-> oracle state conversion."""
from __future__ import annotations

import numpy as np
import torch

from oracle import struprune_oracle as O

# Tolerances for values (weights, auxiliary variables, accumulators):
#   bf16 GEMM inputs with fp32 accumulation: 2e-3;  fp32 mode: 1e-5   (max |x - y| / max |y| per tensor).
TOL = {torch.bfloat16: 2e-3, torch.float32: 1e-5}


def relerr(x, y) -> float:
    """max_ij |x - y| / max_ij |y|."""
    x = np.asarray(x, np.float64)
    y = np.asarray(y, np.float64)
    den = np.abs(y).max() if y.size else 0.0
    if den == 0.0:
        return float(np.abs(x).max()) if x.size else 0.0
    return float(np.abs(x - y).max() / den)


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def bf16_half_ulp(y: np.ndarray) -> np.ndarray:
    """Half a bf16 unit in the last place at |y| (bound of one round-to-nearest to bf16)."""
    a = np.abs(y)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    return np.where(a > 0, 2.0 ** (e - 8), 0.0)


def oracle_state_from_gpu(mod) -> O.FfnState:
    """Snapshot of the GPU module's state as an oracle state (paper orientation: tokens are columns)."""
    return O.FfnState(
        Z=np64(mod.Z).T.copy(), U=None if mod.U is None else np64(mod.U).T.copy(), G_X=np64(mod.G_X),
        G_A=np64(mod.G_A), R1=np64(mod.R1), R2=np64(mod.R2), absA=np64(mod.absA), mask=mod.mask.cpu().numpy().copy())


def lower(G: np.ndarray) -> np.ndarray:
    return np.tril(G)
