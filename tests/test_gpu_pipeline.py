"""Algorithm 1 end to end on a tiny three-layer model: importances, softmax-form allocation, per-layer ADMM loops, all
through the C ABI, checked against the oracle step by step (the oracle is fed the GPU's importances for the
allocation, and each layer's first iteration is compared like the single-module tests)."""
import numpy as np
import pytest
import torch

from oracle import struprune_oracle as O
from paper_2510_03246_b200 import api, pipeline, synth
from tests._util import TOL, np64, relerr

pytestmark = pytest.mark.gpu
DEV = "cuda"
CFG = synth.scaled(synth.CONFIGS["C1"], layers=3, d=96, n=328, tokens=600)


def _inputs(layer):
    X = synth.make_activations(CFG, layer)
    W1, W2 = synth.make_weights(CFG, layer)
    # make the layers differ in scale so that the allocation is not uniform
    return X.to(DEV), (W1 * (1.0 + 0.5 * layer)).to(DEV), (W2 * (1.0 + 0.25 * layer)).to(DEV)


def test_algorithm1_three_layers():
    rbar, iters = 0.5, 2
    p = api.AdmmParams(rho=CFG.rho)
    results, r, k_keep, timing = pipeline.prune_ffn_layers(_inputs, CFG.layers, CFG.n, rbar, iters, params=p)
    assert len(results) == CFG.layers and timing["layers_per_s"] > 0
    # Step 1: layer importances against the oracle on the same inputs
    I_gpu = np.array([res.importance for res in results])
    for l, res in enumerate(results):
        X, W1, W2 = _inputs(l)
        st, _ = O.ffn_init(np64(X).T, np64(W1), np64(W2))
        _, I_or = O.wanda_scores(np64(W2), colsq=np.diag(st.G_A), kind="l2")
        assert abs(res.importance - I_or) < TOL[torch.float32] * abs(I_or) * 10
    # Step 2: allocation from the GPU's importances, fp64 on both sides
    T = float(np.abs(I_gpu).mean())
    r_or, k_or = O.allocate_sparsity(I_gpu, [CFG.n] * CFG.layers, rbar, T)
    assert np.abs(np64(r) - r_or).max() < 1e-12
    assert np.array_equal(k_keep.cpu().numpy(), k_or)
    assert abs(r_or.sum() - rbar * CFG.layers) < 1e-9          # nothing clipped: the budget holds with equality
    assert len(set(k_or.tolist())) > 1                           # and the allocation is not uniform here
    # Steps 3/4: every layer ends with exactly its kept count, pruned rows / columns zero, residuals reported
    for l, res in enumerate(results):
        m = res.mask.cpu().numpy()
        assert int(m.sum()) == int(k_or[l]) == res.k_keep
        assert np.all(np64(res.W1)[m == 0] == 0) and np.all(np64(res.W2)[:, m == 0] == 0)
        assert len(res.reports) == iters and all(rep["kept"] == res.k_keep for rep in res.reports)
        assert all(np.isfinite(rep["res_act"]) and rep["res_act"] >= 0 for rep in res.reports)


def test_temperature_search_matches_oracle_losses():
    """Outer loop of Algorithm 1: for every temperature of the grid the total loss L(T) = sum_l L_l (Step 5) equals
    what the oracle gets by running Steps 1-5 itself on the same inputs, and both pick the same T*.  fp32 mode, two
    free-running iterations per layer: every tensor of a step agrees to 1e-5 (max relative error), the loss is a sum of
    squares of such tensors over two steps, so it is compared to 2e-4 relative."""
    grid = [0.25, 1.0, 4.0]
    iters, rbar = 2, 0.5
    best, losses, results = pipeline.temperature_search(_inputs, CFG.layers, CFG.n, rbar, iters, grid,
                                                        params=api.AdmmParams(rho=CFG.rho))
    layers = []
    for l in range(CFG.layers):
        X, W1, W2 = _inputs(l)
        layers.append((np64(X).T, np64(W1), np64(W2)))
    want, kept = {}, {}
    for T_rel in grid:
        want[T_rel], _, _, kept[T_rel] = O.temperature_loss(layers, rbar, T_rel, iters, O.AdmmParams(rho=CFG.rho))
        assert abs(losses[T_rel] - want[T_rel]) <= 2e-4 * want[T_rel], (T_rel, losses[T_rel], want[T_rel])
    assert len({round(v, 6) for v in want.values()}) == len(grid)      # the temperatures give different losses here
    assert best == min(want, key=want.get)
    # the layers returned are those of the best temperature, with the kept counts the oracle allocates at it
    assert [res.k_keep for res in results] == [max(1, int(k)) for k in kept[best]]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_attention_head_pruning_matches_oracle(dtype):
    """Head scores, top-k heads and the W_O recovery on the kept heads, composed from the library calls, against the
    same composition of oracle functions."""
    N, d, H = 900, 96, 8
    dh = d // H
    Hout = (synth.standard_variates(71, 1, N * d, "gauss").view(N, d)).to(dtype)
    scale = 0.2 + synth.standard_variates(71, 5, H, "gauss").abs().repeat_interleave(dh)      # heads of unequal weight
    Wo = (synth.standard_variates(71, 2, d * d, "gauss").view(d, d) * 0.1 * scale[None, :]).float()
    Ypre = (Hout.float() @ Wo.T).to(dtype)
    k = 5
    mask, W_new, scores = pipeline.prune_attention_heads(Hout.to(DEV), Ypre.to(DEV), Wo.to(DEV), H, k, rho=0.1,
                                                         token_chunk=400)
    tol = 1e-5 if dtype == torch.float32 else 2e-3
    Hd, Yd, Wd = np64(Hout.float()).T, np64(Ypre.float()).T, np64(Wo)
    G = Hd @ Hd.T
    R = Yd @ Hd.T
    s_or, _ = O.wanda_scores(Wd, colsq=np.diag(G), kind="l2", group=dh)
    assert relerr(np64(scores), s_or) < tol
    m_ref, _ = O.topk_mask(scores.cpu().numpy(), k)          # the integer decision in the GPU's precision
    assert np.array_equal(mask.cpu().numpy(), m_ref) and int(mask.sum()) == k
    keep_cols = np.repeat(mask.cpu().numpy(), dh)
    ref = O.restricted_refit(R, G, keep_cols, O.effective_ridge(G, 0.1, True))
    assert relerr(np64(W_new), ref) < tol
    assert np.all(np64(W_new)[:, keep_cols == 0] == 0.0)


@pytest.mark.parametrize("bf16", [False, True])
def test_fixed_mask_continuation_on_kept_channels(bf16):
    """After the mask is fixed, the iterations continue on the kept channels only.  Checked two ways: against the
    oracle run on the reduced module (teacher-forced from the compact state), and against the full-width module
    stepped with the same fixed mask (absolute ridge, so that both solve the same systems)."""
    import copy
    from tests._util import oracle_state_from_gpu
    cfg = synth.scaled(synth.CONFIGS["C2" if bf16 else "C1"], d=136, n=520, tokens=900, sparsity=0.5, outlier_frac=0.02)
    X = synth.make_activations(cfg, 0).to(DEV)
    W1, W2 = (w.to(DEV) for w in synth.make_weights(cfg, 0))
    tol = TOL[X.dtype]
    k = cfg.k_keep
    full = api.FfnModule(X, W1, W2)
    full.sp_ffn_init()
    p_sel = api.AdmmParams(k_keep=k, rho=0.05, rho_relative=False)
    full.sp_admm_step(p_sel)                                   # this step selects the mask
    comp, idx = pipeline.compact_module(full)
    assert int(idx.numel()) == k and torch.equal(full.mask.nonzero().flatten(), idx)
    p_fix_full = api.AdmmParams(k_keep=k, rho=0.05, rho_relative=False, reselect_mask=False, skip_scores=True)
    p_fix_comp = api.AdmmParams(k_keep=k, rho=0.05, rho_relative=False, reselect_mask=False, skip_scores=True)
    for it in range(2):
        # oracle on the reduced module, restarted from the compact state
        st = oracle_state_from_gpu(comp)
        st.mask = np.ones(k, np.uint8)
        p_or = O.AdmmParams(k_keep=k, rho=0.05, rho_relative=False, reselect_mask=False)
        Xo, Yo = np64(X).T, np64(comp.Ypre).T
        comp.sp_admm_step(p_fix_comp)
        full.sp_admm_step(p_fix_full)
        torch.cuda.synchronize()
        comp.check_status(); full.check_status()
        O.admm_step(st, Xo, Yo, np64(comp.W1_0), p_or)
        assert relerr(np64(comp.W1), st.W1) < tol and relerr(np64(comp.W2), st.W2) < tol
        assert relerr(np64(comp.Z).T, st.Z) < tol
        assert relerr(np64(comp.G_A), st.G_A) < tol and relerr(np64(comp.R1), st.R1) < tol
        # the full-width module with the same fixed mask walks the same path on the kept channels
        W1e, W2e = pipeline.expand_weights(comp, idx, cfg.n)
        assert relerr(np64(W1e), np64(full.W1)) < 2 * tol and relerr(np64(W2e), np64(full.W2)) < 2 * tol
        assert relerr(np64(comp.Z), np64(full.Z[:, idx])) < 2 * tol
    # skip_scores needs a fixed mask and the recovery on the kept support
    with pytest.raises(api.SpError) as e:
        full.sp_admm_step(api.AdmmParams(k_keep=k, skip_scores=True))
    assert e.value.code == 1


@pytest.mark.parametrize("kind,bf16", [("wanda_l2", False), ("lemma1", False), ("wanda_l2", True)])
def test_lockstep_global_threshold(kind, bf16):
    """Appendix B, Algorithm 3 (GSPO) in lock step over three layers: per iteration the scores of all layers, one
    global threshold, then every layer's recovery and a-/z-updates with the mask it was given.  The oracle walks the
    same loop on its own from the same inputs (fp32 case: masks must agree bit for bit and the final weights within
    tolerance); the last selection is also checked against the oracle's threshold on the GPU's own scores."""
    import copy
    cfg = synth.scaled(synth.CONFIGS["C2" if bf16 else "C1"], layers=3, d=96, n=328, tokens=600, outlier_frac=0.02)
    kinds = {"wanda_l2": api.SP_SCORE_WANDA_L2, "lemma1": api.SP_SCORE_LEMMA1}

    def inputs(layer):
        X = synth.make_activations(cfg, layer)
        W1, W2 = synth.make_weights(cfg, layer)
        return X.to(DEV), (W1 * (1.0 + 0.5 * layer)).to(DEV), (W2 * (1.0 + 0.25 * layer)).to(DEV)

    L, n, keep, iters = cfg.layers, cfg.n, 0.4, 2
    p = api.AdmmParams(rho=cfg.rho, score_kind=kinds[kind])
    results, scores, masks = pipeline.prune_ffn_layers_global(inputs, L, n, keep, iters, params=p, token_chunk=256)
    torch.cuda.synchronize()
    K = int(keep * n * L + 1e-9)
    m_gpu = masks.cpu().numpy()
    assert m_gpu.sum() == K and [r.k_keep for r in results] == m_gpu.sum(axis=1).tolist()
    # the integer decision in the GPU's precision: the oracle's threshold on the GPU's scores of the last iteration
    m_ref, counts_ref, _ = O.global_threshold_masks(scores.cpu().numpy(), keep, min_keep=1)
    assert np.array_equal(m_gpu, m_ref)
    assert len(set(counts_ref.tolist())) > 1                    # the layers end with different kept counts
    for l, res in enumerate(results):
        mk = m_gpu[l]
        assert np.array_equal(res.mask.cpu().numpy(), mk)
        assert np.all(np64(res.W1)[mk == 0] == 0) and np.all(np64(res.W2)[:, mk == 0] == 0)
        assert [rep["kept"] for rep in res.reports] and res.reports[-1]["kept"] == mk.sum()
    # the oracle's own lock-step run
    tol = TOL[torch.bfloat16 if bf16 else torch.float32]
    p_or = O.AdmmParams(rho=cfg.rho, score_kind=kind)
    states, data = [], []
    for l in range(L):
        X, W1, W2 = inputs(l)
        st, Y = O.ffn_init(np64(X).T, np64(W1), np64(W2))
        states.append(st)
        data.append((np64(X).T, Y, np64(W1)))
    agree = True
    for it in range(iters):
        S = np.stack([O.admm_weight_phase(copy.deepcopy(st), data[l][2], p_or, cfg.tokens)[0]
                      for l, st in enumerate(states)])
        m_or, counts, _ = O.global_threshold_masks(S, keep, min_keep=1)
        for l, st in enumerate(states):
            st.mask = m_or[l].copy()
            pl = copy.deepcopy(p_or)
            pl.reselect_mask, pl.k_keep = False, int(counts[l])
            O.admm_step(st, data[l][0], data[l][1], data[l][2], pl)
    S_gpu = scores.cpu().numpy().astype(np.float64)
    assert relerr(S_gpu, S) < tol * 10                           # scores after one full iteration of every layer
    diff = np.flatnonzero(m_gpu.reshape(-1) != m_or.reshape(-1))
    if diff.size:                                                # only units within rounding of the threshold may differ
        tau = np.sort(S.reshape(-1))[::-1][K - 1]
        assert np.all(np.abs(S.reshape(-1)[diff] - tau) <= 10 * tol * np.abs(S).max())
        agree = False
    if not bf16:
        assert agree
    if agree:
        for l, res in enumerate(results):
            assert relerr(np64(res.W1), states[l].W1) < tol * 10, l
            assert relerr(np64(res.W2), states[l].W2) < tol * 10, l
