"""Parity of the attention-module path (sp_mha_init, sp_mha_step) with the oracle's Method-2 functions (Appendix A,
"Computation on Multi-Head Attention layers"; Algorithm 2, SparseLLM2) at reduced size, in fp32 and bf16 mode, through
the C ABI.  The oracle works on one sequence with tokens as columns; the library stores everything token-major."""
import numpy as np
import pytest
import torch

from oracle import struprune_oracle as O
from paper_2510_03246_b200 import api, synth
from tests._util import TOL, bf16_half_ulp, np64, relerr

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(dtype, d, H, T, n_seq, seed_layer=0):
    cfg = synth.scaled(synth.CONFIGS["C2"], d=d, tokens=n_seq * T, outlier_frac=0.0,
                       storage="f32" if dtype == torch.float32 else "bf16")
    X = synth.make_activations(cfg, seed_layer)
    ws = []
    for tid in (11, 12, 13, 14):
        w = synth.standard_variates(synth.module_seed(cfg, seed_layer), tid, d * d, "gauss").view(d, d)
        ws.append((w * (1.2 / np.sqrt(d))).to(X.dtype))       # projections of unit-scale inputs stay O(1)
    return X, ws


def _oracle_forward(X, W, H, T, n_seq, causal):
    Xo = np64(X)
    out = []
    for q in range(n_seq):
        out.append(O.mha_forward(Xo[q * T:(q + 1) * T].T, *[np64(w) for w in W], H, causal))
    return out


CASES = [(torch.float32, 48, 4, 20, 3, 2, True), (torch.float32, 32, 1, 33, 2, 0, False),
         (torch.bfloat16, 96, 4, 40, 3, 2, True), (torch.bfloat16, 256, 2, 136, 2, 1, False),
         (torch.bfloat16, 128, 2, 264, 1, 0, True), (torch.bfloat16, 512, 8, 520, 2, 1, True),
         # three heads of width 128: three blocks per system in the batched solves of the W_V recovery
         (torch.bfloat16, 384, 3, 72, 2, 1, True)]


@pytest.mark.parametrize("dtype,d,H,T,n_seq,chunk,causal", CASES)
def test_mha_init_matches_forward_definition(dtype, d, H, T, n_seq, chunk, causal):
    X, W = _case(dtype, d, H, T, n_seq)
    mod = api.MhaModule(X.to(DEV), *[w.to(DEV) for w in W], n_heads=H, T=T, seq_chunk=chunk)
    mod.sp_mha_init(causal)
    torch.cuda.synchronize()
    mod.check_status()
    tol = TOL[dtype]
    ref = _oracle_forward(X, W, H, T, n_seq, causal)
    for q, (Zq, Zk, V, P, A, Y) in enumerate(ref):
        r = slice(q * T, (q + 1) * T)
        assert relerr(np64(mod.Zq[r]).T, Zq) < tol and relerr(np64(mod.Zk[r]).T, Zk) < tol
        assert relerr(np64(mod.P[q]), P) < tol, "P"
        assert relerr(np64(mod.Aattn[r]).T, A) < tol, "Aattn"
        got = np64(mod.Ypre[r]).T
        if dtype == torch.bfloat16:
            assert np.all(np.abs(got - Y) <= tol * np.abs(Y).max() + bf16_half_ulp(Y) * 1.001)
        else:
            assert relerr(got, Y) < tol


@pytest.mark.parametrize("dtype,d,H,T,n_seq,chunk,causal", CASES)
def test_mha_step_teacher_forced(dtype, d, H, T, n_seq, chunk, causal):
    """Three outer steps with pruned weights (one head removed, the others perturbed); before every step the oracle
    restarts from the GPU's state, then both take the step: Eq. (85) gradient steps on P, Eq. (86) closed form,
    Eq. (87) gradient steps on (Zq, Zk)."""
    X, W = _case(dtype, d, H, T, n_seq, seed_layer=1)
    mod = api.MhaModule(X.to(DEV), *[w.to(DEV) for w in W], n_heads=H, T=T, seq_chunk=chunk)
    mod.sp_mha_init(causal)
    dh = d // H
    Wp = [w.float().clone() for w in W]
    if H > 1:
        for w in Wp[:3]:
            w[:dh] = 0
        Wp[3][:, :dh] = 0
    g = torch.Generator().manual_seed(7)
    for w in Wp:
        w.mul_(1.0 + 0.05 * torch.randn(w.shape, generator=g))
    mod.set_weights(*[w.to(DEV) for w in Wp])
    p_gpu = api.MhaParams(alpha=0.8, beta=1.3, a_steps=3, z_steps=2, eta_z=0.9, causal=causal)
    p_or = O.MhaParams(n_heads=H, alpha=0.8, beta=1.3, a_steps=3, z_steps=2, eta_z=0.9, causal=causal)
    tol = TOL[dtype]
    Xo, Yo = np64(X), None
    Wo64 = [np64(w) for w in Wp]
    for it in range(3):
        torch.cuda.synchronize()
        before = [np64(t) for t in (mod.Zq, mod.Zk, mod.P, mod.Aattn)]
        Yo = np64(mod.Ypre)
        mod.sp_mha_step(p_gpu)
        torch.cuda.synchronize()
        mod.check_status()
        obj0 = obj1 = 0.0
        for q in range(n_seq):
            r = slice(q * T, (q + 1) * T)
            st = (before[0][r].T, before[1][r].T, before[2][q], before[3][r].T)
            Zq, Zk, P, A = O.mha_step(Xo[r].T, Yo[r].T, *Wo64, *st, p_or)
            assert relerr(np64(mod.P[q]), P) < tol, ("P", it, q)
            assert relerr(np64(mod.Aattn[r]).T, A) < tol, ("Aattn", it, q)
            assert relerr(np64(mod.Zq[r]).T, Zq) < tol and relerr(np64(mod.Zk[r]).T, Zk) < tol, ("Z", it, q)
            obj0 += O.mha_objective(Xo[r].T, Yo[r].T, *Wo64, *st, p_or).sum()
            got = (np64(mod.Zq[r]).T, np64(mod.Zk[r]).T, np64(mod.P[q]), np64(mod.Aattn[r]).T)
            obj1 += O.mha_objective(Xo[r].T, Yo[r].T, *Wo64, *got, p_or).sum()
        assert obj1 < obj0            # the GPU's new state lowers the Method-2 objective


def test_mha_argument_errors():
    X, W = _case(torch.bfloat16, 96, 4, 40, 2)
    mod = api.MhaModule(X.to(DEV), *[w.to(DEV) for w in W], n_heads=4, T=40)
    mod.sp_mha_init()
    with pytest.raises(api.SpError) as e:
        mod.sp_mha_step(api.MhaParams(alpha=-1.0))
    assert e.value.code == 1
    with pytest.raises(api.SpError) as e:
        mod.sp_mha_step(api.MhaParams(eta_z=2.0))
    assert e.value.code == 1
    with pytest.raises(api.SpError) as e:          # head width 20 is not a multiple of 8: no 16-byte aligned slices
        api.MhaModule(X[:, :80].contiguous().to(DEV), *[w[:80, :80].contiguous().to(DEV) for w in W], n_heads=4,
                      T=40).sp_mha_init()
    assert e.value.code == 4


@pytest.mark.parametrize("dtype,d,H,T,n_seq", [(torch.float32, 48, 4, 20, 3), (torch.bfloat16, 128, 4, 72, 3)])
def test_mha_outer_iterations_match_oracle(dtype, d, H, T, n_seq):
    """Two outer iterations of SparseLLM2 with one head pruned, teacher-forced per iteration: the accumulators the
    module holds, the projections recovered from them (W_Q, W_K by ridge solves with masked rows, W_O on the kept heads)
    and the auxiliary updates that follow, each against the oracle restarted from the GPU's state."""
    from paper_2510_03246_b200 import pipeline
    X, W = _case(dtype, d, H, T, n_seq, seed_layer=2)
    mod = api.MhaModule(X.to(DEV), *[w.to(DEV) for w in W], n_heads=H, T=T, seq_chunk=2)
    mod.sp_mha_init(True)
    dh = d // H
    head_mask = torch.ones(H, dtype=torch.uint8)
    head_mask[1] = 0
    hm = head_mask.to(DEV)
    p_gpu = api.MhaParams(alpha=1.0, beta=1.2, a_steps=2, z_steps=2, causal=True)
    p_or = O.MhaParams(n_heads=H, alpha=1.0, beta=1.2, a_steps=2, z_steps=2, causal=True)
    tol = TOL[dtype]
    Xo = np64(X)
    Xs = [Xo[q * T:(q + 1) * T].T for q in range(n_seq)]
    Wv_masked = np64(W[2].float()).copy()
    Wv_masked[dh:2 * dh] = 0
    for it in range(2):
        torch.cuda.synchronize()
        Yo = np64(mod.Ypre)
        seqs = lambda t: [np64(t)[q * T:(q + 1) * T].T for q in range(n_seq)]
        Zqs, Zks, As, Ys = seqs(mod.Zq), seqs(mod.Zk), seqs(mod.Aattn), [Yo[q * T:(q + 1) * T].T for q in range(n_seq)]
        Ps = [np64(mod.P[q]) for q in range(n_seq)]
        # accumulators left by the previous call
        assert relerr(np64(mod.G_X), sum(x @ x.T for x in Xs)) < tol
        assert relerr(np64(mod.R_Q), sum(z @ x.T for z, x in zip(Zqs, Xs))) < tol
        assert relerr(np64(mod.R_K), sum(z @ x.T for z, x in zip(Zks, Xs))) < tol
        assert relerr(np64(mod.G_attn), sum(a @ a.T for a in As)) < tol
        assert relerr(np64(mod.R_O), sum(y @ a.T for y, a in zip(Ys, As))) < tol
        acc = {k: np64(getattr(mod, k)) for k in ("G_X", "R_Q", "R_K", "G_attn", "R_O")}
        # first iteration with the row-masked pre-trained W_V, second with W_V recovered from P and Aattn
        pipeline.mha_outer_iterations(mod, hm, 1, p_gpu, rho=0.1, recover_wv=(it == 1))
        torch.cuda.synchronize()
        # weights: the oracle's recovery from the GPU's accumulators (teacher-forced)
        keep = np.repeat(head_mask.numpy().astype(bool), dh)
        rho1 = O.effective_ridge(acc["G_X"], 0.1, True)
        Wq_or = np.where(keep[:, None], O.ridge_solve(acc["R_Q"], acc["G_X"], rho1), 0.0)
        Wk_or = np.where(keep[:, None], O.ridge_solve(acc["R_K"], acc["G_X"], rho1), 0.0)
        Wo_or = O.restricted_refit(acc["R_O"], acc["G_attn"], keep, O.effective_ridge(acc["G_attn"], 0.1, True))
        assert relerr(np64(mod.Wq), Wq_or) < tol and relerr(np64(mod.Wk), Wk_or) < tol, "W_Q / W_K"
        assert relerr(np64(mod.Wo), Wo_or) < tol, "W_O"
        assert np.all(np64(mod.Wq)[~keep] == 0) and np.all(np64(mod.Wo)[:, ~keep] == 0) and np.all(np64(mod.Wv)[~keep] == 0)
        if it == 0:
            assert relerr(np64(mod.Wv), Wv_masked) < 1e-7
        else:
            Wv_or = O.mha_recover_value_weights(Xs, Ps, As, head_mask.numpy(), dh, 0.1, True)
            assert relerr(np64(mod.Wv), Wv_or) < tol, "W_V"
        # auxiliary updates with the GPU's weights
        Wg = [np64(w) for w in (mod.Wq, mod.Wk, mod.Wv, mod.Wo)]
        for q in range(n_seq):
            r = slice(q * T, (q + 1) * T)
            Zq, Zk, P, A = O.mha_step(Xs[q], Ys[q], *Wg, Zqs[q], Zks[q], Ps[q], As[q], p_or)
            assert relerr(np64(mod.P[q]), P) < tol and relerr(np64(mod.Aattn[r]).T, A) < tol
            assert relerr(np64(mod.Zq[r]).T, Zq) < tol and relerr(np64(mod.Zk[r]).T, Zk) < tol


@pytest.mark.parametrize("dtype,d,H,T,n_seq,chunk,causal", CASES)
def test_mha_value_refit_matches_oracle(dtype, d, H, T, n_seq, chunk, causal):
    """W_V = a_attn (P X)^+ per kept head (sp_mha_value_refit) against the oracle's recovery from the same P, Aattn, X,
    after one step with perturbed weights (so that P and Aattn are no longer the forward values): with a relative
    ridge and one head pruned, then with all heads and an absolute ridge written into a pitched output."""
    X, W = _case(dtype, d, H, T, n_seq, seed_layer=3)
    mod = api.MhaModule(X.to(DEV), *[w.to(DEV) for w in W], n_heads=H, T=T, seq_chunk=chunk)
    mod.sp_mha_init(causal)
    g = torch.Generator().manual_seed(9)
    Wp = [w.float() * (1.0 + 0.05 * torch.randn(w.shape, generator=g)) for w in W]
    mod.set_weights(*[w.to(DEV) for w in Wp])
    mod.sp_mha_step(api.MhaParams(alpha=1.0, beta=1.0, a_steps=2, z_steps=1, causal=causal))
    torch.cuda.synchronize()
    mod.check_status()
    dh = d // H
    tol = TOL[dtype]
    Xo = np64(X)
    Xs = [Xo[q * T:(q + 1) * T].T for q in range(n_seq)]
    As = [np64(mod.Aattn)[q * T:(q + 1) * T].T for q in range(n_seq)]
    Ps = [np64(mod.P[q]) for q in range(n_seq)]
    head_mask = [1] * H
    if H > 1:
        head_mask[H // 2] = 0
    Wv = mod.sp_mha_value_refit(head_mask, 0.05, True)
    torch.cuda.synchronize()
    mod.check_status()
    ref = O.mha_recover_value_weights(Xs, Ps, As, head_mask, dh, 0.05, True)
    assert relerr(np64(Wv), ref) < tol
    keep = np.repeat(np.asarray(head_mask, bool), dh)
    assert np.all(np64(Wv)[~keep] == 0)
    # all heads, absolute ridge, output rows 8 floats apart from a dense layout; the padding is not touched
    out = torch.full((d, d + 8), -3.0, device=DEV)
    rho_abs = 0.02 * float(np.trace(sum(x @ x.T for x in Xs))) / d
    mod.sp_mha_value_refit(None, rho_abs, False, out=out[:, :d])
    torch.cuda.synchronize()
    mod.check_status()
    ref2 = O.mha_recover_value_weights(Xs, Ps, As, [1] * H, dh, rho_abs, False)
    assert relerr(np64(out[:, :d]), ref2) < tol
    assert torch.all(out[:, d:] == -3.0)


def test_mha_value_refit_argument_errors():
    X, W = _case(torch.bfloat16, 96, 4, 40, 2)
    mod = api.MhaModule(X.to(DEV), *[w.to(DEV) for w in W], n_heads=4, T=40)
    mod.sp_mha_init()
    with pytest.raises(api.SpError) as e:
        mod.sp_mha_value_refit(None, -1.0, True)
    assert e.value.code == 1
    m, st = mod._module(), mod._state()
    import ctypes as C
    rc = api.lib().sp_mha_value_refit(C.byref(m), C.byref(st), None, 0.1, 1, 0, mod.Wv.data_ptr(), mod.d,
                                      mod.status.data_ptr(), mod._wsbuf.data_ptr(), 256, None)
    assert rc == 5                                   # SP_ERR_WORKSPACE
    rc = api.lib().sp_mha_value_refit(C.byref(m), C.byref(st), None, 0.1, 1, 0, mod.Wv.data_ptr(), mod.d - 8,
                                      mod.status.data_ptr(), mod._wsbuf.data_ptr(), mod._wsbuf.numel(), None)
    assert rc == 2                                   # SP_ERR_SHAPE: leading dimension below d
