"""Pins of the oracle's multi-head-attention path (Appendix A, "Computation on Multi-Head Attention layers", Method 2;
Algorithm 2, SparseLLM2).  The paper prints no numbers for it, so every check is against mathematics that does not
depend on the oracle's own formulas: central differences of the objectives, the definition of the module written as
plain loops, stationarity / optimality of each sub-step, and special cases that reduce to linear algebra."""
import math

import numpy as np
import pytest

from oracle import struprune_oracle as O


def _module(seed, d=8, T=6, h=2, scale=0.6):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((d, T))
    W = [scale * rng.standard_normal((d, d)) for _ in range(4)]
    return X, W


def test_forward_matches_loop_definition():
    """head_i = softmax(Q_i^T K_i / sqrt(d_h)) applied to V_i, concatenated, times W_O -- token by token."""
    X, (Wq, Wk, Wv, Wo) = _module(1)
    d, T = X.shape
    h, dh = 2, 4
    for causal in (False, True):
        Zq, Zk, V, P, A, Y = O.mha_forward(X, Wq, Wk, Wv, Wo, h, causal)
        Q, K, Vv = Wq @ X, Wk @ X, Wv @ X
        A_ref = np.zeros((d, T))
        for i in range(h):
            for t in range(T):
                keys = range(t + 1) if causal else range(T)
                logit = {u: sum(Q[i * dh + c, t] * K[i * dh + c, u] for c in range(dh)) / math.sqrt(dh) for u in keys}
                mx = max(logit.values())
                den = sum(math.exp(v - mx) for v in logit.values())
                for u in keys:
                    w = math.exp(logit[u] - mx) / den
                    assert P[i, t, u] == pytest.approx(w, rel=1e-12)
                    for c in range(dh):
                        A_ref[i * dh + c, t] += w * Vv[i * dh + c, u]
                assert P[i, t].sum() == pytest.approx(1.0)
                if causal:
                    assert np.all(P[i, t, t + 1:] == 0.0)
        assert np.allclose(A, A_ref, atol=1e-13) and np.allclose(Y, Wo @ A_ref, atol=1e-12)
        # at the pre-trained weights and the initial auxiliary variables every term of the objective vanishes
        p = O.MhaParams(n_heads=h, causal=causal)
        assert np.all(O.mha_objective(X, Y, Wq, Wk, Wv, Wo, Zq, Zk, P, A, p) < 1e-24)


def _central(f, x, eps=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        old = x[idx]
        x[idx] = old + eps; fp = f()
        x[idx] = old - eps; fm = f()
        x[idx] = old
        g[idx] = (fp - fm) / (2 * eps)
    return g


def test_gradients_against_central_differences():
    rng = np.random.default_rng(2)
    dh, T = 4, 5
    alpha, beta = 0.7, 1.3
    for causal in (False, True):
        # Eq. (85): gradient in P
        P, Phi = rng.random((T, T)), O.softmax_rows(rng.standard_normal((T, T)), causal)
        A_i, V_i = rng.standard_normal((dh, T)), rng.standard_normal((dh, T))
        _, g = O.mha_a_objective_grad(P, A_i, V_i, Phi, alpha, beta)
        g_fd = _central(lambda: O.mha_a_objective_grad(P, A_i, V_i, Phi, alpha, beta)[0], P)
        assert np.allclose(g, g_fd, atol=1e-6)
        # Eq. (87): gradients in Zq and Zk through the softmax
        Zq, Zk = rng.standard_normal((dh, T)), rng.standard_normal((dh, T))
        Tq, Tk = rng.standard_normal((dh, T)), rng.standard_normal((dh, T))
        Pt = O.softmax_rows(rng.standard_normal((T, T)), causal)
        f = lambda: O.mha_z_objective_grad(Zq, Zk, Pt, Tq, Tk, alpha, beta, causal)[0]
        _, gq, gk = O.mha_z_objective_grad(Zq, Zk, Pt, Tq, Tk, alpha, beta, causal)
        assert np.allclose(gq, _central(f, Zq), atol=1e-6) and np.allclose(gk, _central(f, Zk), atol=1e-6)
        # the objective of Eq. (87) is what the full objective's terms 3-5 say for one head
        p = O.MhaParams(n_heads=1, alpha=alpha, beta=beta, causal=causal)
        I = np.eye(dh)
        terms = O.mha_objective(np.eye(dh, T), np.zeros((dh, T)), I, I, I, I, Zq, Zk, Pt[None], np.zeros((dh, T)), p)
        f87 = O.mha_z_objective_grad(Zq, Zk, Pt, np.eye(dh, T), np.eye(dh, T), alpha, beta, causal)[0]
        assert terms[2:].sum() == pytest.approx(f87, rel=1e-12)


def test_attn_update_is_the_minimiser_of_eq86():
    X, (Wq, Wk, Wv, Wo) = _module(3)
    rng = np.random.default_rng(4)
    Y, Hd = rng.standard_normal(X.shape), rng.standard_normal(X.shape)
    A = O.mha_attn_update(Y, Wo, Hd)
    grad = -2 * Wo.T @ (Y - Wo @ A) + 2 * (A - Hd)
    assert np.abs(grad).max() < 1e-11
    f = lambda A_: ((Y - Wo @ A_) ** 2).sum() + ((A_ - Hd) ** 2).sum()
    for _ in range(5):
        assert f(A + 1e-3 * rng.standard_normal(A.shape)) > f(A)
    # W_O = 0: the output term is constant and a^attn equals the head outputs
    assert np.allclose(O.mha_attn_update(Y, np.zeros_like(Wo), Hd), Hd)


def test_every_substep_descends_and_the_a_steps_converge():
    """After pruning (rows of W_Q, W_K, W_V and columns of W_O of one head zeroed) each of the three updates lowers
    the Method-2 objective, for several seeds; the gradient steps of Eq. (85), a strictly convex quadratic taken with
    the step 1 / L, converge to its minimiser, which a linear solve gives directly."""
    for seed in range(6):
        X, (Wq, Wk, Wv, Wo) = _module(10 + seed, d=12, T=9, h=3, scale=0.8)
        h, dh = 3, 4
        for causal in (False, True):
            Zq, Zk, V0, P, A, Y = O.mha_forward(X, Wq, Wk, Wv, Wo, h, causal)
            Wq2, Wk2, Wv2, Wo2 = Wq.copy(), Wk.copy(), Wv.copy(), Wo.copy()
            Wq2[:dh] = 0; Wk2[:dh] = 0; Wv2[:dh] = 0; Wo2[:, :dh] = 0
            Wv2[dh:] *= 0.9
            p = O.MhaParams(n_heads=h, alpha=0.8, beta=1.1, a_steps=3, z_steps=3, causal=causal)
            obj = lambda st: O.mha_objective(X, Y, Wq2, Wk2, Wv2, Wo2, *st, p).sum()
            st = (Zq, Zk, P, A)
            V = Wv2 @ X
            for _ in range(3):
                f0 = obj(st)
                P1 = O.mha_a_update(st[2], st[3], V, st[0], st[1], p)
                f1 = obj((st[0], st[1], P1, st[3]))
                A1 = O.mha_attn_update(Y, Wo2, O.mha_heads(V, P1, h))
                f2 = obj((st[0], st[1], P1, A1))
                Zq1, Zk1 = O.mha_z_update(st[0], st[1], P1, Wq2 @ X, Wk2 @ X, p)
                f3 = obj((Zq1, Zk1, P1, A1))
                assert f1 <= f0 + 1e-12 and f2 <= f1 + 1e-12 and f3 <= f2 + 1e-12
                full = O.mha_step(X, Y, Wq2, Wk2, Wv2, Wo2, *st, p)
                assert all(np.array_equal(a, b) for a, b in zip(full, (Zq1, Zk1, P1, A1)))
                st = full
    # convergence of the a-steps to the minimiser of Eq. (85) for one head: P (alpha V^T V + beta I) = alpha A^T V + beta Phi
    rng = np.random.default_rng(5)
    dh, T = 3, 5
    V_i, A_i = 0.5 * rng.standard_normal((dh, T)), rng.standard_normal((dh, T))
    Zq_i, Zk_i = rng.standard_normal((dh, T)), rng.standard_normal((dh, T))
    p = O.MhaParams(n_heads=1, alpha=0.6, beta=1.4, a_steps=4000, causal=False)
    Phi = O.softmax_rows(O.mha_logits(Zq_i, Zk_i))
    P_inf = O.mha_a_update(rng.random((1, T, T)), A_i, V_i, Zq_i, Zk_i, p)[0]
    P_star = np.linalg.solve(p.alpha * V_i.T @ V_i + p.beta * np.eye(T), (p.alpha * A_i.T @ V_i + p.beta * Phi).T).T
    assert np.allclose(P_inf, P_star, atol=1e-9)


def test_special_cases():
    """One token: the softmax of a single logit is 1, so the module is the linear map W_O W_V and, with the weights
    unchanged, a step leaves the initial state where it is.  One head with very sharp logits (queries equal to keys,
    scaled up): the probabilities approach the identity and the head output approaches V."""
    rng = np.random.default_rng(6)
    d = 6
    x = rng.standard_normal((d, 1))
    W = [rng.standard_normal((d, d)) for _ in range(4)]
    Zq, Zk, V, P, A, Y = O.mha_forward(x, *W, 2)
    assert np.all(P == 1.0) and np.allclose(Y, W[3] @ W[2] @ x)
    p = O.MhaParams(n_heads=2)
    st = O.mha_step(x, Y, *W, Zq, Zk, P, A, p)
    assert np.allclose(st[0], Zq) and np.allclose(st[1], Zk) and np.allclose(st[2], P) and np.allclose(st[3], A)
    T = 5
    Xs = 8.0 * np.linalg.qr(rng.standard_normal((d, d)))[0][:, :T]        # orthogonal columns, large norm
    I = np.eye(d)
    _, _, V, P, A, _ = O.mha_forward(Xs, I, I, W[2], I, 1, causal=False)
    assert np.abs(P[0] - np.eye(T)).max() < 1e-9 and np.allclose(A, V, atol=1e-7)
    # the step of Eq. (87) shrinks with the size of the iterate and never exceeds the step of its quadratic part
    assert O.mha_z_step_size(Xs, Xs, 1.0, 1.0, 1.0) < O.mha_z_step_size(0.1 * Xs, 0.1 * Xs, 1.0, 1.0, 1.0) < 0.5


def test_recovered_projections_reproduce_the_pretrained_ones_and_respect_the_head_mask():
    """W = z a^+ for the projections that are linear in the auxiliary variables: from the pre-trained state, all heads
    kept and a vanishing ridge, the recoveries return W_Q, W_K, W_O (X and the head outputs have full row rank over the
    sequences); with a head removed its rows of W_Q, W_K and its columns of W_O are zero, the other rows of W_Q, W_K
    are unchanged, and the kept columns of W_O are the least-squares fit on those columns alone."""
    rng = np.random.default_rng(8)
    d, T, h, dh, n_seq = 8, 9, 2, 4, 3
    W = [0.7 * rng.standard_normal((d, d)) for _ in range(4)]
    Xs = [rng.standard_normal((d, T)) for _ in range(n_seq)]
    fw = [O.mha_forward(X, *W, h, True) for X in Xs]
    Zqs, Zks, As, Ys = [f[0] for f in fw], [f[1] for f in fw], [f[4] for f in fw], [f[5] for f in fw]
    Wq, Wk, Wo = O.mha_recover_weights(Xs, Ys, Zqs, Zks, As, [1, 1], dh, 1e-12, False)
    assert np.allclose(Wq, W[0], atol=1e-8) and np.allclose(Wk, W[1], atol=1e-8) and np.allclose(Wo, W[3], atol=1e-7)
    Wq1, Wk1, Wo1 = O.mha_recover_weights(Xs, Ys, Zqs, Zks, As, [0, 1], dh, 1e-12, False)
    assert np.all(Wq1[:dh] == 0) and np.all(Wk1[:dh] == 0) and np.all(Wo1[:, :dh] == 0)
    assert np.allclose(Wq1[dh:], W[0][dh:], atol=1e-8) and np.allclose(Wk1[dh:], W[1][dh:], atol=1e-8)
    A_all, Y_all = np.concatenate(As, axis=1), np.concatenate(Ys, axis=1)
    fit = np.linalg.lstsq(A_all[dh:].T, Y_all.T, rcond=None)[0].T          # Ypre ~ W_O[:, kept] Aattn[kept]
    assert np.allclose(Wo1[:, dh:], fit, atol=1e-7)


def test_recovered_value_projection():
    """W_V = a^attn (X P^T)^+ per head.  Pins: (1) from the pre-trained state with a vanishing ridge it returns W_V (the
    regressors X P_i^T of three sequences have full row rank); (2) the result is the minimiser of the second term of the
    Method 2 objective plus the ridge: central differences of that term, evaluated by O.mha_objective, vanish there
    and every perturbation raises it; (3) one token per sequence (P = 1): the regressors are X itself and the recovery is
    the plain ridge solve on G_X, as lstsq on the stacked system gives it; (4) rows of a pruned head are zero and the
    other heads do not change (the heads' systems are separate)."""
    rng = np.random.default_rng(11)
    d, T, h, dh, n_seq = 8, 9, 2, 4, 3
    W = [0.7 * rng.standard_normal((d, d)) for _ in range(4)]
    Xs = [rng.standard_normal((d, T)) for _ in range(n_seq)]
    fw = [O.mha_forward(X, *W, h, True) for X in Xs]
    Ps, As = [f[3] for f in fw], [f[4] for f in fw]
    Wv = O.mha_recover_value_weights(Xs, Ps, As, [1, 1], dh, 1e-13, False)
    assert np.allclose(Wv, W[2], atol=1e-6)
    # (2) perturbed auxiliary variables, a real ridge: stationarity of  sum_s |A_s - heads(Wv X_s, P_s)|^2 + rho |Wv|^2
    As2 = [A + 0.3 * rng.standard_normal(A.shape) for A in As]
    Ps2 = [np.abs(P + 0.05 * rng.standard_normal(P.shape)) for P in Ps]
    rho = 0.37
    Wv2 = O.mha_recover_value_weights(Xs, Ps2, As2, [1, 1], dh, rho, False)
    prm = O.MhaParams(n_heads=h, alpha=1.0, beta=1.0)

    def f(Wtry):
        t2 = sum(O.mha_objective(X, np.zeros((d, T)), W[0], W[1], Wtry, W[3], np.zeros((d, T)), np.zeros((d, T)), P, A,
                                 prm)[1] for X, P, A in zip(Xs, Ps2, As2))
        return t2 + rho * (Wtry ** 2).sum()

    f0 = f(Wv2)
    eps = 1e-5
    for (i, j) in [(0, 0), (3, 5), (4, 1), (7, 7)]:
        E = np.zeros((d, d)); E[i, j] = eps
        assert abs(f(Wv2 + E) - f(Wv2 - E)) / (2 * eps) < 1e-6 * max(f0, 1.0)
    for _ in range(5):
        assert f(Wv2 + 1e-3 * rng.standard_normal((d, d))) > f0
    # (3) T = 1: softmax of one logit is 1
    X1 = [rng.standard_normal((d, 1)) for _ in range(20)]
    A1 = [rng.standard_normal((d, 1)) for _ in range(20)]
    P1 = [np.ones((h, 1, 1)) for _ in range(20)]
    Wv3 = O.mha_recover_value_weights(X1, P1, A1, [1, 1], dh, 1e-13, False)
    Xa, Aa = np.concatenate(X1, axis=1), np.concatenate(A1, axis=1)
    assert np.allclose(Wv3, np.linalg.lstsq(Xa.T, Aa.T, rcond=None)[0].T, atol=1e-7)
    # relative ridge: rho times the mean diagonal of the head's own Gram matrix
    G0 = sum((X @ P[0].T) @ (X @ P[0].T).T for X, P in zip(Xs, Ps2))
    C0 = sum(A[:dh] @ (X @ P[0].T).T for X, P, A in zip(Xs, Ps2, As2))
    Wrel = O.mha_recover_value_weights(Xs, Ps2, As2, [1, 1], dh, 0.1, True)
    assert np.allclose(Wrel[:dh], C0 @ np.linalg.inv(G0 + 0.1 * np.trace(G0) / d * np.eye(d)), atol=1e-9)
    # (4) head mask
    Wv4 = O.mha_recover_value_weights(Xs, Ps2, As2, [0, 1], dh, rho, False)
    assert np.all(Wv4[:dh] == 0) and np.array_equal(Wv4[dh:], Wv2[dh:])
