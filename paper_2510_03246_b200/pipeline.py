"""Model-level flow of Algorithm 1 ("Importance-Guided Global Structured Pruning") over the FFN modules of a model,
built from the library calls only (argument marshalling and loop control; all arithmetic runs in libsp).

    Step 1  layer importances I_l        sp_ffn_init + sp_struct_scores on the pre-trained module
    Step 2  softmax-form allocation      sp_allocate_sparsity  (r_l -> kept units per layer)
    Step 3/4 per-module ADMM             sp_admm_step x K with the layer's kept count
    Step 5  loss L(T) = sum_l L_l        the module objectives reported by the last step (temperature_search)

plan_distribute covers Steps 1 and 2 of the "-distribute" variant (importances from weight statistics, attention and
MLP modules allocated separately by inverse weighting).

One module is resident at a time (the paper's memory argument), so a layer is initialised twice: once for its
importance, once for its ADMM loop.  With several ranks each rank owns the layers `parallel.layers_of_rank` gives it;
the only exchange is the vector of importances before Step 2.
"""
from __future__ import annotations

import time
from dataclasses import dataclass, field
from typing import Callable

import torch

from . import api, parallel


@dataclass
class LayerResult:
    layer: int
    importance: float
    k_keep: int
    mask: torch.Tensor            # u8 [n]
    W1: torch.Tensor              # fp32 [n, d]
    W2: torch.Tensor              # fp32 [d, n]
    reports: list = field(default_factory=list)
    last_report: torch.Tensor | None = None    # device copy of the last step's report


def layer_importance(X, W1_0, W2_0, score_kind=api.SP_SCORE_WANDA_L2, token_chunk=0) -> float:
    """I_l of one pre-trained FFN module: mean unit score of W2_0 against the pre-trained activation statistics."""
    mod = api.FfnModule(X, W1_0, W2_0, token_chunk=token_chunk)
    mod.sp_ffn_init()
    n = mod.n
    if score_kind == api.SP_SCORE_WANDA_L2:
        _, imp, _ = api.sp_struct_scores(score_kind, n, W=mod.W2_0, colsq=mod.G_A, colsq_stride=n + 1)
    elif score_kind == api.SP_SCORE_WANDA_L1:
        _, imp, _ = api.sp_struct_scores(score_kind, n, W=mod.W2_0, colabs=mod.absA, inv_tokens=1.0 / mod.N)
    else:
        raise ValueError("layer importance uses one of the Wanda score kinds")
    mod.check_status()
    return float(imp.item())


def layer_importances(layer_inputs, n_layers, score_kind=api.SP_SCORE_WANDA_L2, token_chunk=0, device="cuda"):
    """Step 1 of Algorithm 1 for all layers (each rank its own, then gathered): fp64 [n_layers] on the device."""
    rank, _, world = parallel.env_world()
    local = {}
    for l in parallel.layers_of_rank(n_layers, rank, world):
        X, W1_0, W2_0 = layer_inputs(l)
        local[l] = layer_importance(X, W1_0, W2_0, score_kind, token_chunk)
    return parallel.gather_importances(local, n_layers, device=device).to(device)


def prune_ffn_layers(layer_inputs: Callable[[int], tuple], n_layers: int, n_units: int, rbar: float, iters: int,
                     params: api.AdmmParams | None = None, T_rel: float = 1.0, alloc_mode=api.SP_ALLOC_SOFTMAX,
                     token_chunk: int = 0, device="cuda", planned=None):
    """Runs Algorithm 1 over `n_layers` FFN modules.  layer_inputs(l) returns (X [N, d], W1_0 [n, d], W2_0 [d, n]) on the
    device for layer l.  planned = (I_all, r, k_keep) skips Steps 1 and 2 (the outer temperature loop computes the
    importances once and the allocations of its whole grid in one launch).
    Returns (results of the layers this rank owns, r per layer, kept counts per layer, timings)."""
    rank, _, world = parallel.env_world()
    mine = parallel.layers_of_rank(n_layers, rank, world)
    p = params or api.AdmmParams()
    t0 = time.perf_counter()
    if planned is None:
        I_all = layer_importances(layer_inputs, n_layers, p.score_kind, token_chunk, device)       # Step 1
        # Step 2 (the temperature is given relative to the magnitude of the importances; the library scales it)
        nu = torch.full((n_layers,), n_units, dtype=torch.int64, device=device)
        T_list = torch.tensor([float(T_rel)], dtype=torch.float64, device=device)
        r, k_keep = api.sp_allocate_sparsity_grid(I_all, nu, rbar, T_list, True, alloc_mode)
        r, k_keep = r[0], k_keep[0]
    else:
        I_all, r, k_keep = planned
    k_host = k_keep.cpu().tolist()
    t1 = time.perf_counter()
    # Steps 3 and 4
    results = []
    for l in mine:
        X, W1_0, W2_0 = layer_inputs(l)
        k = max(1, int(k_host[l]))
        mod = api.FfnModule(X, W1_0, W2_0, dual_mode=p.dual_mode, token_chunk=token_chunk, overlap_k=k)
        mod.sp_ffn_init()
        pl = api.AdmmParams(**{**p.__dict__, "k_keep": k, "token_chunk": token_chunk})
        res = LayerResult(l, float(I_all[l].item()), k, None, None, None)
        for _ in range(iters):
            mod.sp_admm_step(pl)
            res.reports.append(mod.report.clone())
        mod.check_status()
        res.mask, res.W1, res.W2 = mod.mask.clone(), mod.W1.clone(), mod.W2.clone()
        res.last_report = res.reports[-1] if res.reports else None
        res.reports = [dict(zip(api.REPORT_FIELDS, t.cpu().tolist())) for t in res.reports]
        results.append(res)
        del mod
    torch.cuda.synchronize()
    t2 = time.perf_counter()
    return results, r, k_keep, {"importance_s": t1 - t0, "admm_s": t2 - t1, "layers_per_s": len(mine) / max(t2 - t0, 1e-9)}


def prune_ffn_layers_global(layer_inputs: Callable[[int], tuple], n_layers: int, n_units: int, keep_fraction: float,
                            iters: int, params: api.AdmmParams | None = None, token_chunk: int = 0, min_keep: int = 1,
                            device="cuda"):
    """Lock-step run of Appendix B, Algorithm 3 (GSPO): in every iteration the scores of ALL layers are computed from
    their current states, ONE threshold over the concatenated scores keeps K = floor(keep_fraction * n_units *
    n_layers) units of the whole model, and every layer finishes the iteration (recovery on its kept support, a- and
    z-updates) with the mask it was given.  The states of all layers stay resident (Z alone is N x n fp32 per layer);
    the modules share one workspace.  min_keep: a layer the threshold leaves with fewer units keeps its own min_keep
    best ones (sp_admm_step needs at least one).  Returns (results per layer, scores [L, n], masks [L, n])."""
    p = params or api.AdmmParams()
    L, n = n_layers, n_units
    scores = torch.zeros(L, n, dtype=torch.float32, device=device)
    masks = torch.ones(L, n, dtype=torch.uint8, device=device)
    pool, mods = {}, []
    overlap_k = min(n, int(1.5 * keep_fraction * n) + 1)
    for l in range(L):
        X, W1_0, W2_0 = layer_inputs(l)
        mod = api.FfnModule(X, W1_0, W2_0, dual_mode=p.dual_mode, token_chunk=token_chunk, overlap_k=overlap_k,
                            scores=scores[l], mask=masks[l], ws_pool=pool)
        mod.sp_ffn_init()
        mods.append(mod)
    results = [LayerResult(l, float("nan"), 0, None, None, None) for l in range(L)]
    p_scores = api.AdmmParams(**{**p.__dict__, "k_keep": 1, "token_chunk": token_chunk, "skip_scores": False})
    for _ in range(iters):
        for mod in mods:
            mod.sp_admm_scores(p_scores)
        # one threshold over all layers, the repair of emptied layers and the kept counts: one library call
        _, _, kept = api.sp_apply_mask_global(scores, keep_fraction, min_keep, mask_out=masks)
        counts = kept.cpu().tolist()                      # kept units per layer: host arguments of the calls below
        for l, mod in enumerate(mods):
            # with the recovery on the kept support nothing of the unrestricted recovery is needed again
            pl = api.AdmmParams(**{**p.__dict__, "k_keep": int(counts[l]), "token_chunk": token_chunk,
                                   "reselect_mask": False, "skip_scores": bool(p.refit)})
            mod.sp_admm_step(pl)
            results[l].reports.append(mod.report.clone())
            results[l].k_keep = int(counts[l])
    for l, mod in enumerate(mods):
        mod.check_status()
        res = results[l]
        res.importance = float(mod.importance.item())
        res.mask, res.W1, res.W2 = mod.mask.clone(), mod.W1.clone(), mod.W2.clone()
        res.reports = [dict(zip(api.REPORT_FIELDS, t.cpu().tolist())) for t in res.reports]
    return results, scores, masks


def compact_module(mod: api.FfnModule):
    """Continuation of a module whose mask is fixed (the flow of Algorithm 1, where Step 3 fixes the masks before the
    SparseLLM iterations): a new module that holds only the kept channels.  With a fixed mask the pruned channels
    never enter a kept channel's updates again (their columns of W2 and rows of W1 are zero), so the iterations can
    go on at width k instead of n: accumulators k x k instead of n x n, no unrestricted recovery, no scores.
    Pure data movement (gathers); returns (compact module, kept channel indices).  Run it with
    AdmmParams(k_keep=k, reselect_mask=False, skip_scores=True); with rho_relative the ridge of the W2 recovery is
    then relative to the trace over the kept channels only."""
    idx = torch.nonzero(mod.mask, as_tuple=False).flatten()
    k = int(idx.numel())
    new = api.FfnModule(mod.X, mod.W1_0[idx], mod.W2_0[:, idx], dual_mode=mod.U is not None,
                        token_chunk=mod.token_chunk, overlap_k=k, Wg_0=mod.Wg_0[idx] if mod.Wg_0 is not None else None)
    new.Ypre = mod.Ypre
    new.Z.copy_(mod.Z[:, idx])
    if mod.U is not None:
        new.U.copy_(mod.U[:, idx])
    if mod.Gate is not None:
        new.Gate.copy_(mod.Gate[:, idx])
    new.G_X = mod.G_X
    new.G_A.copy_(mod.G_A[idx][:, idx])
    new.R1.copy_(mod.R1[idx])
    new.R2.copy_(mod.R2[:, idx])
    new.absA.copy_(mod.absA[idx])
    new.mask.fill_(1)
    new.iteration = mod.iteration
    return new, idx


def expand_weights(cmod: api.FfnModule, idx: torch.Tensor, n: int):
    """W1 [n, d] and W2 [d, n] of the full module from a compact continuation (pruned rows / columns zero)."""
    W1 = torch.zeros(n, cmod.d, dtype=torch.float32, device=cmod.dev)
    W2 = torch.zeros(cmod.d, n, dtype=torch.float32, device=cmod.dev)
    W1[idx] = cmod.W1
    W2[:, idx] = cmod.W2
    return W1, W2


def prune_attention_heads(H: torch.Tensor, Ypre: torch.Tensor, W_O: torch.Tensor, n_heads: int, k_heads: int,
                          rho: float = 0.1, token_chunk: int = 32768):
    """Head pruning of one attention module with its head outputs held fixed (Algorithm 2, attention branch, W_O part;
    Algorithm 1 Step 3 with heads as units).  H [N, d]: concatenated head outputs (the input of the output
    projection), Ypre [N, d]: the pre-trained module output, W_O [d, d] fp32.  Head h owns columns
    [h d_head, (h + 1) d_head) of W_O.  Steps, all library calls:
      G_H = H^T H, R = Ypre^T H          sp_gram_accumulate over token chunks
      head scores                       sp_struct_scores, Wanda-l2 over the head's column block of W_O
      keep the k_heads best             sp_apply_mask
      W_O[:, S] = R[:, S](G_H[S,S] + rho_eff I)^-1, other heads zero     sp_linear_refit (ridge of the full system)
    Returns (mask u8 [n_heads], W_O_new fp32 [d, d], scores fp32 [n_heads])."""
    N, d = H.shape
    d_head = d // n_heads
    G = torch.zeros(d, d, dtype=torch.float32, device=H.device)
    R = torch.zeros(d, d, dtype=torch.float32, device=H.device)
    for t0 in range(0, N, token_chunk):
        api.sp_gram_accumulate(H[t0:t0 + token_chunk], Ypre[t0:t0 + token_chunk], G, R)
    api.sp_symmetrize(G)
    scores, _, _ = api.sp_struct_scores(api.SP_SCORE_WANDA_L2, n_heads, d_head, W=W_O, colsq=G, colsq_stride=d + 1)
    mask, _, _ = api.sp_apply_mask(scores, k_heads)
    W_new = api.sp_linear_refit(R, G, mask, k_heads, rho, group=d_head, rho_relative=True)
    return mask, W_new, scores


def mha_outer_iterations(mod: api.MhaModule, head_mask: torch.Tensor, iters: int, params: api.MhaParams | None = None,
                         rho: float = 0.1, rho_relative: bool = True, recover_wv: bool = True):
    """Outer loop of Algorithm 2's SparseLLM2 for one attention module with a fixed head mask (u8 [n_heads], from the
    head scores): per iteration (1) the weight recoveries W = z a^+ "for W_Q, W_K, W_V, W_O separately" -- W_Q, W_K by
    sp_ridge_solve from the accumulators the previous step left, with the rows of pruned heads zeroed, W_O by
    sp_linear_refit on the columns of the kept heads, W_V by sp_mha_value_refit from P and Aattn (one system per kept
    head; recover_wv = False keeps the row-masked pre-trained W_V instead) -- then (2) sp_mha_step: Eq. (85), (86),
    (87).  `mod` must have been initialised (sp_mha_init) with its accumulators.
    All arithmetic runs in the library; this function only orders the calls.  Returns the module."""
    p = params or api.MhaParams()
    d_head = mod.d // mod.n_heads
    k_heads = int(head_mask.sum().item())
    mask_host = head_mask.cpu().tolist()
    # row masks of the projections: sp_apply_mask zeroes the rows of pruned units given their scores; with the mask
    # already known its 0 / 1 values serve as the scores and k_heads as the kept count
    unit_scores = head_mask.to(torch.float32)
    api.sp_apply_mask(unit_scores, k_heads, group=d_head, W_rows=mod.Wv)
    precise = mod.X.dtype == torch.float32          # fp32 mode: fp64 factorisations
    for _ in range(iters):
        Wq = api.sp_ridge_solve(mod.R_Q, mod.G_X, rho, rho_relative, precise)
        Wk = api.sp_ridge_solve(mod.R_K, mod.G_X, rho, rho_relative, precise)
        api.sp_apply_mask(unit_scores, k_heads, group=d_head, W_rows=Wq)
        api.sp_apply_mask(unit_scores, k_heads, group=d_head, W_rows=Wk)
        Wo = api.sp_linear_refit(mod.R_O, mod.G_attn, head_mask, k_heads, rho, group=d_head, precise=precise,
                                 rho_relative=rho_relative)
        if recover_wv:
            mod.sp_mha_value_refit(mask_host, rho, rho_relative)      # writes mod.Wv, rows of pruned heads zero
        mod.set_weights(Wq, Wk, mod.Wv, Wo)
        mod.sp_mha_step(p)
    mod.check_status()
    return mod


def plan_distribute(layer_weights: Callable[[int], dict], n_layers: int, n_heads: int, n_ffn: int, rbar: float,
                    T_rel: float = 1.0, rho: float = 1.0, gamma: float = 1.0, device="cuda"):
    """Steps 1 and 2 of the "-distribute" variant of Algorithm 1: importances of the attention and MLP modules from
    weight statistics (with depth decay gamma^l and the attention/MLP ratio rho), normalised separately, turned into
    pruned fractions by the inverse weighting.  layer_weights(l) returns dict(Wq, Wk, Wv, Wo, fc1, fc2) on the device
    for layer l (one layer resident at a time).  Returns dict(I_attn, I_mlp, r_attn, r_mlp, k_heads, k_channels)."""
    head_stats = torch.zeros(n_layers, n_heads, 4, dtype=torch.float64, device=device)
    fc_stats = torch.zeros(n_layers, 2, 4, dtype=torch.float64, device=device)
    for l in range(n_layers):
        w = layer_weights(l)
        d_head = w["Wq"].shape[0] // n_heads
        for name in ("Wq", "Wk", "Wv"):            # head h = rows [h d_head, (h + 1) d_head)
            api.sp_weight_stats(w[name], 0, d_head, head_stats[l], accumulate=True)
        api.sp_weight_stats(w["Wo"], 1, d_head, head_stats[l], accumulate=True)   # and the same columns of W_O
        api.sp_weight_stats(w["fc1"], 0, 0, fc_stats[l, 0:1])
        api.sp_weight_stats(w["fc2"], 0, 0, fc_stats[l, 1:2])
    I_attn, I_mlp = api.sp_distribute_importance(head_stats, fc_stats, rho, gamma)
    out = {"I_attn": I_attn, "I_mlp": I_mlp}
    for key, I, units in (("attn", I_attn, n_heads), ("mlp", I_mlp, n_ffn)):
        T = T_rel * float(I.abs().mean())
        nu = torch.full((n_layers,), units, dtype=torch.int64, device=device)
        r, k = api.sp_allocate_sparsity(I, nu, rbar, T, api.SP_ALLOC_INVERSE)
        out["r_" + key] = r
        out["k_heads" if key == "attn" else "k_channels"] = k
    return out


def total_loss(results, beta: float, device="cuda") -> float:
    """L(T) = sum_l L_l of Algorithm 1 Step 5 over the given layers: the FFN objective of Appendix A.1 after each
    layer's last iteration, summed on the device (needs compute_objective in the parameters)."""
    loss = torch.zeros(1, dtype=torch.float64, device=device)
    for res in results:
        api.sp_objective_accumulate(res.last_report, beta, loss, True)
    return float(loss.item())


def temperature_search(layer_inputs: Callable[[int], tuple], n_layers: int, n_units: int, rbar: float, iters: int,
                       T_grid, params: api.AdmmParams | None = None, **kw):
    """Outer loop of Algorithm 1: run the whole flow for every relative temperature of `T_grid` and keep the one with
    the smallest total loss.  Returns (best T_rel, {T_rel: loss summed over this rank's layers}, results at the best T).
    With several ranks the losses are summed over ranks before the comparison."""
    p = params or api.AdmmParams()
    p = api.AdmmParams(**{**p.__dict__, "compute_objective": True})
    device = kw.get("device", "cuda")
    # Steps 1 and 2 do not depend on the iterations: importances once, the allocations of the whole grid in one launch
    I_all = layer_importances(layer_inputs, n_layers, p.score_kind, kw.get("token_chunk", 0), device)
    nu = torch.full((n_layers,), n_units, dtype=torch.int64, device=device)
    T_list = torch.tensor([float(t) for t in T_grid], dtype=torch.float64, device=device)
    r_all, k_all = api.sp_allocate_sparsity_grid(I_all, nu, rbar, T_list, True, kw.get("alloc_mode", api.SP_ALLOC_SOFTMAX))
    losses, best = {}, None
    for g, T_rel in enumerate(T_grid):
        results, r, k_keep, _ = prune_ffn_layers(layer_inputs, n_layers, n_units, rbar, iters, params=p, T_rel=T_rel,
                                                 planned=(I_all, r_all[g], k_all[g]), **kw)
        loss = parallel.sum_over_ranks(total_loss(results, p.beta, kw.get("device", "cuda")), device=kw.get("device", "cuda"))
        losses[float(T_rel)] = loss
        if best is None or loss < best[1]:
            best = (float(T_rel), loss, results, r, k_keep)
    return best[0], losses, best[2]
