"""Multi-GPU plumbing: the per-module path shards over independent modules (layers), one process per GPU.

Once the kept counts are fixed, every module's ADMM loop is independent, so ranks own disjoint sets of layers and the
data path needs no collective.  The only cross-rank exchange is the vector of layer importances (L doubles) that the
sparsity allocation reads, gathered once before the loops start.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment (1 process if unset)."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def layers_of_rank(n_layers: int, rank: int, world: int) -> list[int]:
    """Round-robin assignment of layer indices to ranks (balanced within one layer)."""
    return list(range(rank, n_layers, world))


def gather_importances(local: dict[int, float], n_layers: int, device="cpu") -> torch.Tensor:
    """All ranks contribute the importances of the layers they own; every rank gets the full fp64 vector."""
    vec = torch.zeros(n_layers, dtype=torch.float64, device=device)
    for layer, val in local.items():
        vec[layer] = val
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(vec, op=dist.ReduceOp.SUM)
    return vec


def max_over_ranks(value: float, device="cpu") -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
