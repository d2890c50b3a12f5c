"""Multi-GPU plumbing, one process per GPU.

Sharding over modules: once the kept counts are fixed, every module's ADMM loop is independent, so ranks own disjoint
sets of layers and the data path needs no collective.  The only cross-rank exchange is the vector of layer importances
(L doubles) that the sparsity allocation reads, gathered once before the loops start.

Sharding over tokens inside ONE module (`token_sharded_iterations`): the a-, z- and dual updates are local to a token,
and the weight recovery sees the tokens only through the accumulators G_X, G_A, R1, R2 (and the column sums of |A|),
which are sums over tokens.  Every rank therefore keeps its token shard of X, Ypre, Z, U, repeats the (small) weight
phase on the summed accumulators, and the only exchange per iteration is one all-reduce of the accumulators its token
pass produced — into each GPU's own memory, before any kernel reads them — plus a broadcast of the n-byte mask so that
rounding differences between ranks cannot make them select different units.
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


ACCUMULATORS = ("G_A", "R1", "R2", "absA")      # rebuilt by every token pass; G_X is a sum over tokens of the inputs only
N_REPORT_SUMS = 5     # res_act, res_out, res_in, z_sq, a_sq: sums over tokens; the other report fields are not


def _dist_on():
    return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1


def _sum_shards(shards, name):
    """Sum of the tensor `name` over the local shards and over the ranks, written back to every shard."""
    ts = [getattr(m, name) for m in shards]
    total = ts[0]
    for t in ts[1:]:
        total.add_(t)
    if _dist_on():
        dist.all_reduce(total, op=dist.ReduceOp.SUM)
    for t in ts[1:]:
        t.copy_(total)


def token_sharded_init(shards):
    """Initialisation of one module whose tokens are split over `shards`: every shard initialises its own tokens, then
    the accumulators are summed.  `shards`: the module objects of this process — one per process under
    torch.distributed, several only when one process stands in for several (tests)."""
    for m in shards:
        m.sp_ffn_init()
    for name in ("G_X",) + ACCUMULATORS:
        _sum_shards(shards, name)


def token_sharded_iterations(shards, params, iters: int, read_reports: bool = True):
    """`iters` ADMM iterations of one module over token shards.  Per iteration: every shard computes the unit scores
    from the (identical) summed accumulators; rank 0's first shard selects the mask and everyone adopts it; every shard
    finishes the iteration on its own tokens with that mask; the new accumulators are summed.  `params` as for
    sp_admm_step (k_keep, score kind, ...).  Returns the per-iteration reports (token sums added over all shards) as
    dicts, or with read_reports = False as device tensors (no host synchronisation inside the loop).
    The l1 score kind divides by a shard's own token count: masks are unaffected, its layer importance is scaled by
    the number of shards when they are of equal size."""
    import copy
    p_scores = copy.copy(params)
    p_scores.skip_scores, p_scores.reselect_mask = False, True
    p_fixed = copy.copy(params)
    p_fixed.reselect_mask = False
    p_fixed.skip_scores = bool(params.refit)
    reports = []
    for _ in range(iters):
        for m in shards:
            m.sp_admm_scores(p_scores)
        if params.reselect_mask:
            lead = shards[0]
            lead.select_mask(params.k_keep)
            if _dist_on():
                dist.broadcast(lead.mask, src=0)
            for m in shards[1:]:
                m.mask.copy_(lead.mask)
        for m in shards:
            m.sp_admm_step(p_fixed)
        for name in ACCUMULATORS:
            _sum_shards(shards, name)
        # token sums of the step report (the first fields of the report vector) over shards and ranks, on the device
        rep = shards[0].report.clone()
        for m in shards[1:]:
            rep[:N_REPORT_SUMS] += m.report[:N_REPORT_SUMS]
        if _dist_on():
            dist.all_reduce(rep[:N_REPORT_SUMS], op=dist.ReduceOp.SUM)
        reports.append(rep)
    if not read_reports:
        return reports
    names = shards[0].report_fields
    reports = [dict(zip(names, r.cpu().tolist())) for r in reports]
    return reports
