"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test checks an oracle function against something other than itself: a hand-evaluated value stored
under tests/golden/, a closed form, an invariant, a textbook library routine of a different kind
(pinv / lstsq / full sort), or brute force on tiny inputs.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import struprune_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- Gram / cross products
def test_gram_matches_triple_loop_and_identities():
    r = _rng(1)
    d, m, N = 5, 3, 7
    X = r.normal(size=(d, N))
    Y = r.normal(size=(m, N))
    G = np.zeros((d, d)); R = np.zeros((m, d)); st = np.zeros((d, 2))
    # two chunks, to exercise accumulation
    O.gram_accumulate(G, R, X[:, :4], Y[:, :4], st)
    O.gram_accumulate(G, R, X[:, 4:], Y[:, 4:], st)
    Gb = np.zeros((d, d)); Rb = np.zeros((m, d))
    for i in range(d):
        for j in range(d):
            for t in range(N):
                Gb[i, j] += X[i, t] * X[j, t]
    for i in range(m):
        for j in range(d):
            for t in range(N):
                Rb[i, j] += Y[i, t] * X[j, t]
    assert np.allclose(G, Gb, rtol=1e-13, atol=1e-13)
    assert np.allclose(R, Rb, rtol=1e-13, atol=1e-13)
    assert np.allclose(G, G.T)
    assert np.isclose(np.trace(G), sum(np.dot(X[:, t], X[:, t]) for t in range(N)))
    assert np.allclose(st[:, 1], np.diag(G))
    assert np.allclose(st[:, 0], [sum(abs(X[i, t]) for t in range(N)) for i in range(d)])


# ---------------------------------------------------------------- ridge solve / recovery
def test_ridge_identity_input_closed_form():
    r = _rng(2)
    R = r.normal(size=(4, 6))
    W = O.ridge_solve(R, np.eye(6), 0.25)
    assert np.allclose(W, R / 1.25, rtol=1e-14)


def test_ridge_normal_equations_and_pinv_limit():
    r = _rng(3)
    d, n, N = 6, 4, 40
    X = r.normal(size=(d, N))
    Z = r.normal(size=(n, N))
    G = X @ X.T
    R = Z @ X.T
    rho = 0.3
    W = O.ridge_solve(R, G, rho)
    # stationarity of |Z - W X|^2 + rho |W|^2
    grad = (W @ X - Z) @ X.T + rho * W
    assert np.abs(grad).max() < 1e-10
    # rho -> 0 with X of full row rank: W = Z X^+ (Appendix A.1)
    W0 = O.ridge_solve(R, G, 0.0)
    assert np.allclose(W0, Z @ np.linalg.pinv(X), rtol=1e-9, atol=1e-11)
    # perturbing the solution can only increase the regularised objective
    J = lambda W_: ((Z - W_ @ X) ** 2).sum() + rho * (W_ ** 2).sum()
    for _ in range(5):
        assert J(W + 1e-3 * r.normal(size=W.shape)) > J(W)


def test_effective_ridge():
    G = np.diag([1.0, 2.0, 3.0, 6.0])
    assert O.effective_ridge(G, 0.5, True) == pytest.approx(0.5 * 12.0 / 4.0)
    assert O.effective_ridge(G, 0.5, False) == 0.5


def test_restricted_refit_is_least_squares_on_support():
    r = _rng(4)
    n, d, N = 7, 3, 30
    A = r.normal(size=(n, N))
    Y = r.normal(size=(d, N))
    keep = np.array([1, 0, 1, 1, 0, 0, 1], np.uint8)
    S = np.flatnonzero(keep)
    W = O.restricted_refit(Y @ A.T, A @ A.T, keep, 0.0)
    assert np.all(W[:, keep == 0] == 0.0)
    # textbook least squares: min |Y - W_S A_S| solved with lstsq
    Ws = np.linalg.lstsq(A[S].T, Y.T, rcond=None)[0].T
    assert np.allclose(W[:, S], Ws, rtol=1e-9, atol=1e-11)
    # "dense recovery, then refit of its output on the support" gives the same weights as rho -> 0
    Wd = O.ridge_solve(Y @ A.T, A @ A.T, 0.0)
    W2 = np.linalg.lstsq(A[S].T, (Wd @ A).T, rcond=None)[0].T
    assert np.allclose(W[:, S], W2, rtol=1e-8, atol=1e-10)


# ---------------------------------------------------------------- a-update
def test_a_update_stationarity_and_least_squares():
    r = _rng(5)
    n, d, N = 9, 4, 6
    W2 = r.normal(size=(d, n))
    Y = r.normal(size=(d, N))
    Z = r.normal(size=(n, N))
    U = 0.1 * r.normal(size=(n, N))
    alpha, beta = 0.7, 1.9
    for u in (None, U):
        A = O.a_update(W2, Y, Z, alpha, beta, u)
        h = np.maximum(Z, 0) - (0 if u is None else u)
        grad = alpha * W2.T @ (W2 @ A - Y) + beta * (A - h)
        assert np.abs(grad).max() < 1e-11
        # the same minimiser from the stacked least-squares system [sqrt(a) W2; sqrt(b) I] a = [sqrt(a) y; sqrt(b) h]
        M = np.vstack([np.sqrt(alpha) * W2, np.sqrt(beta) * np.eye(n)])
        rhs = np.vstack([np.sqrt(alpha) * Y, np.sqrt(beta) * h])
        assert np.allclose(A, np.linalg.lstsq(M, rhs, rcond=None)[0], rtol=1e-9, atol=1e-11)
        # residual-correction (Woodbury) form with a d x d system: A = h + W2^T (g I + W2 W2^T)^-1 (Y - W2 h)
        C = (beta / alpha) * np.eye(d) + W2 @ W2.T
        assert np.allclose(A, h + W2.T @ np.linalg.solve(C, Y - W2 @ h), rtol=1e-10, atol=1e-12)


def test_a_update_zero_weights_gives_activation():
    r = _rng(6)
    Z = r.normal(size=(5, 3))
    A = O.a_update(np.zeros((2, 5)), r.normal(size=(2, 3)), Z, 1.3, 0.4)
    assert np.allclose(A, np.maximum(Z, 0))


def test_a_update_pruned_columns_keep_activation():
    r = _rng(7)
    n, d, N = 8, 3, 5
    W2 = r.normal(size=(d, n)); W2[:, [1, 4, 6]] = 0.0
    Z = r.normal(size=(n, N))
    A = O.a_update(W2, r.normal(size=(d, N)), Z, 1.0, 1.0)
    assert np.allclose(A[[1, 4, 6]], np.maximum(Z[[1, 4, 6]], 0))


# ---------------------------------------------------------------- z-update
def test_z_candidates_and_paper_rule_hand_cases():
    # one unit, four tokens; W1 X = z1 = [2, -1, 0.5, -3]; a = [1, 1, 0, 2]; alpha = 1, beta = 3
    W1 = np.array([[1.0]])
    X = np.array([[2.0, -1.0, 0.5, -3.0]])
    A = np.array([[1.0, 1.0, 0.0, 2.0]])
    z1, z2 = O.z_candidates(W1, X, A, 1.0, 3.0)
    assert np.allclose(z1, X)
    assert np.allclose(z2, [[(3 * 1 + 2) / 4, (3 * 1 - 1) / 4, (0 + 0.5) / 4, (3 * 2 - 3) / 4]])
    # old z: negative -> z1 ; non-negative (including +0 and -0) -> z2
    Zold = np.array([[-0.1, 0.0, -0.0, 5.0]])
    Zn = O.z_select(Zold, z1, z2, A, 1.0, 3.0, "paper")
    assert np.allclose(Zn, [[2.0, 0.5, 0.125, 0.75]])


def test_z_exact_rule_matches_grid_search():
    r = _rng(8)
    alpha, beta = 0.8, 1.7
    a = r.normal(size=200) * 2
    z1 = r.normal(size=200) * 2
    u = r.normal(size=200) * 0.3
    grid = np.linspace(-12, 12, 480001)
    for use_u in (False, True):
        uu = u if use_u else None
        _, z2 = O.z_candidates(np.eye(1), z1[None, :], a[None, :], alpha, beta, None if uu is None else uu[None, :])
        zn = O.z_select(np.zeros((1, 200)), z1[None, :], z2, a[None, :], alpha, beta, "exact",
                        None if uu is None else uu[None, :])[0]
        for i in range(0, 200, 7):
            ai = a[i] + (u[i] if use_u else 0.0)
            f = beta * (ai - np.maximum(grid, 0)) ** 2 + alpha * (grid - z1[i]) ** 2
            fz = beta * (ai - max(zn[i], 0)) ** 2 + alpha * (zn[i] - z1[i]) ** 2
            assert fz <= f.min() + 1e-9
            assert abs(zn[i] - grid[f.argmin()]) < 1e-3 or abs(fz - f.min()) < 1e-8


def test_dual_update():
    U = np.array([[0.5, -1.0]])
    A = np.array([[2.0, 1.0]])
    Zn = np.array([[1.5, -4.0]])
    assert np.allclose(O.dual_update(U, A, Zn), [[0.5 + 2.0 - 1.5, -1.0 + 1.0 - 0.0]])


# ---------------------------------------------------------------- Lemma 1
def test_lemma1_golden_single_token():
    for ln in _rows("lemma1_cases.txt"):
        b, c, d, t, s = map(float, ln.split())
        sc, rl, e = O.lemma1_scores([[b]], [[c]], [[d]], [[t]])
        assert sc[0] == pytest.approx(s, rel=1e-14, abs=1e-15)
        assert e[0] == pytest.approx(c * c + d * d)
        assert rl == pytest.approx(s)


def test_lemma1_identities():
    r = _rng(9)
    n, N = 12, 9
    c = r.normal(size=(n, N)); d = r.normal(size=(n, N))
    s, rl, e = O.lemma1_scores(c, c, d, d)          # b = c and t = d: nothing is lost, every score is 1
    assert np.allclose(s, 1.0)
    b = r.normal(size=(n, N)); t = r.normal(size=(n, N))
    s, rl, e = O.lemma1_scores(b, c, d, t)
    # s_j is the scalar least-squares coefficient of [b_j; t_j] on [c_j; d_j]
    for j in range(n):
        coef = np.linalg.lstsq(np.concatenate([c[j], d[j]])[:, None], np.concatenate([b[j], t[j]]), rcond=None)[0][0]
        assert s[j] == pytest.approx(coef, rel=1e-10)
    assert rl == pytest.approx(s.sum() / n)
    # groups: numerators and denominators add
    sg, _, eg = O.lemma1_scores(b, c, d, t, group=3)
    num = (c * b).sum(1) + (d * t).sum(1)
    for g in range(n // 3):
        assert sg[g] == pytest.approx(num[3 * g:3 * g + 3].sum() / e[3 * g:3 * g + 3].sum())


def test_relaxed_mask_budget_identity():
    r = _rng(10)
    n = 15
    s = r.normal(size=n); e = r.uniform(0.5, 3.0, size=n)
    for rl in (0.1, 0.5, 0.83):
        M = O.relaxed_mask(s, e, rl)
        assert M.sum() == pytest.approx(rl * n, rel=1e-12)           # the constraint of Eq. (78)
        # stationarity of the Lagrangian: e_j (M_j - s_j) is the same for all j (= -lambda/2)
        lam = e * (M - s)
        assert np.allclose(lam, lam[0])
    assert np.allclose(O.relaxed_mask(s, e, s.mean()), s)            # lambda = 0  <=>  r_l = mean s_j


def test_topk_by_score_is_bruteforce_optimal_for_equal_energies():
    r = _rng(11)
    n, N, k = 10, 4, 4
    c = r.normal(size=(n, N)); d = r.normal(size=(n, N))
    # equalise unit energies e_j = |c_j|^2 + |d_j|^2
    sc = np.sqrt((c * c).sum(1) + (d * d).sum(1))[:, None]
    c /= sc; d /= sc
    b = c + 0.5 * r.normal(size=(n, N)); t = d + 0.5 * r.normal(size=(n, N))
    s, _, e = O.lemma1_scores(b, c, d, t)
    assert np.allclose(e, 1.0)
    mask, tau = O.topk_mask(s, k)

    def loss(m):
        m = np.asarray(m, float)[:, None]
        return ((b - m * c) ** 2).sum() + ((t - m * d) ** 2).sum()

    best = min((loss(np.isin(np.arange(n), S)), S) for S in itertools.combinations(range(n), k))
    assert set(np.flatnonzero(mask)) == set(best[1])
    assert loss(mask) == pytest.approx(best[0])


# ---------------------------------------------------------------- Wanda scores
def test_wanda_scores_definitions():
    r = _rng(12)
    d, n, N = 4, 6, 11
    W = r.normal(size=(d, n)); A = r.normal(size=(n, N))
    s2, I2 = O.wanda_scores(W, colsq=(A * A).sum(1), kind="l2")
    s1, I1 = O.wanda_scores(W, colabs_mean=np.abs(A).mean(1), kind="l1")
    for j in range(n):
        elem = np.abs(W[:, j]) * np.linalg.norm(A[j])           # |W_ij| * |a_j|_2
        assert s2[j] == pytest.approx(np.linalg.norm(elem))
        assert s1[j] == pytest.approx(sum(abs(W[i, j]) * np.abs(A[j]).mean() for i in range(d)))
    assert I2 == pytest.approx(s2.mean()) and I1 == pytest.approx(s1.mean())
    g2, _ = O.wanda_scores(W, colsq=(A * A).sum(1), kind="l2", group=2)
    g1, _ = O.wanda_scores(W, colabs_mean=np.abs(A).mean(1), kind="l1", group=2)
    assert np.allclose(g2, np.sqrt(s2[0::2] ** 2 + s2[1::2] ** 2))
    assert np.allclose(g1, s1[0::2] + s1[1::2])


# ---------------------------------------------------------------- allocation
def test_allocation_golden():
    T = 0.37
    for ln in _rows("allocation_cases.txt"):
        rbar_s, mult_s, r_s = ln.split("|")
        rbar = float(rbar_s)
        I = np.array(list(map(float, mult_s.split()))) * T * np.log(3.0)
        want = np.array(list(map(float, r_s.split())))
        r, k = O.allocate_sparsity(I, [100] * len(I), rbar, T)
        assert np.allclose(r, want, rtol=1e-12)
        assert list(k) == [100 - int(np.floor(100 * w + 0.5)) for w in want]


def test_allocation_invariants():
    r_ = _rng(13)
    L = 24
    I = r_.uniform(0.8, 1.4, size=L)
    nu = np.full(L, 8192)
    r, k = O.allocate_sparsity(I, nu, 0.5, 1.0)
    assert r.sum() == pytest.approx(0.5 * L, rel=1e-12)              # sum r_l = rbar L (Lemma 2)
    assert np.all(np.diff(r[np.argsort(I)]) <= 1e-15)                # low importance -> pruned more
    assert np.all((r >= 0) & (r <= 0.95))
    ru, _ = O.allocate_sparsity(np.full(L, 1.234), nu, 0.5, 0.1)
    assert np.allclose(ru, 0.5)                                      # equal importances -> uniform
    rinf, _ = O.allocate_sparsity(I, nu, 0.5, 1e12)
    assert np.allclose(rinf, 0.5, atol=1e-9)                         # T -> infinity -> uniform
    r0, _ = O.allocate_sparsity(I, nu, 0.5, 1e-4)                    # T -> 0: all mass on argmin I, clipped
    assert r0[np.argmin(I)] == pytest.approx(0.95) and r0.sum() == pytest.approx(0.95)
    assert np.all(k == nu - np.floor(r * nu + 0.5).astype(np.int64))
    rinv, _ = O.allocate_sparsity(I, nu, 0.5, 1.0, mode="inverse")
    assert rinv.sum() == pytest.approx(0.5 * L)
    assert np.all(np.diff(rinv[np.argsort(I)]) >= -1e-15)            # inverse weighting: important -> pruned more
    runi, kuni = O.allocate_sparsity(I, nu, 0.3, 1.0, mode="uniform")
    assert np.allclose(runi, 0.3) and np.all(kuni == 8192 - 2458)


def test_allocation_clip_without_rescale():
    # one layer far less important than the rest: its raw share exceeds 0.95, it is clipped and, because a clip
    # happened, no rescale follows (Algorithm 1 Step 2) -> mass is lost relative to rbar L
    I = np.array([0.0, 5.0, 5.0, 5.0])
    r, _ = O.allocate_sparsity(I, [10] * 4, 0.5, 1.0)
    w = np.exp(-I); w /= w.sum()
    assert r[0] == 0.95 and np.allclose(r[1:], 0.5 * 4 * w[1:])
    assert r.sum() < 0.5 * 4


# ---------------------------------------------------------------- top-k / mask
def test_topk_against_full_sort_and_ties():
    r = _rng(14)
    for n, k in ((1, 1), (17, 0), (17, 17), (257, 100), (1000, 1), (1000, 999)):
        s = np.round(r.normal(size=n), 1)           # coarse rounding creates many exact ties
        mask, tau = O.topk_mask(s, k)
        assert mask.sum() == k
        if 0 < k < n:
            assert s[mask == 1].min() >= s[mask == 0].max()
            assert tau == sorted(s, reverse=True)[k - 1]
            # among units tied at tau the kept ones are the lowest indices
            tied = np.flatnonzero(s == tau)
            kept_t = tied[mask[tied] == 1]
            assert np.array_equal(kept_t, tied[:kept_t.size])
    s = np.array([1.0, np.nan, 3.0, np.nan, 2.0])
    m, tau = O.topk_mask(s, 3)
    assert list(m) == [1, 0, 1, 0, 1]
    m, _ = O.topk_mask(s, 4)
    assert list(m) == [1, 1, 1, 0, 1]


def test_apply_mask_groups():
    W1 = np.arange(24, dtype=float).reshape(6, 4) + 1
    W2 = np.arange(24, dtype=float).reshape(4, 6) + 1
    r_, c_ = O.apply_mask(np.array([1, 0, 1], np.uint8), 2, W_rows=W1, W_cols=W2)
    assert np.all(r_[2:4] == 0) and np.all(r_[:2] == W1[:2]) and np.all(r_[4:] == W1[4:])
    assert np.all(c_[:, 2:4] == 0) and np.all(c_[:, :2] == W2[:, :2]) and np.all(c_[:, 4:] == W2[:, 4:])


# ---------------------------------------------------------------- shapes
def test_opt_shape_table():
    for ln in _rows("opt_shapes.txt"):
        name, d, ffn, mha = ln.split()
        d = int(d)
        n = 4 * d
        assert n * d + d * n == int(ffn) == 8 * d * d
        assert 4 * d * d == int(mha)


# ---------------------------------------------------------------- the loop
def _small_module(seed, d=6, n=12, N=40):
    r = _rng(seed)
    X = r.normal(size=(d, N))
    W1 = r.normal(size=(n, d)) / np.sqrt(d)
    W2 = r.normal(size=(d, n)) / np.sqrt(n)
    return X, W1, W2


def test_init_state_definitions():
    X, W1, W2 = _small_module(20)
    st, Y = O.ffn_init(X, W1, W2)
    Zp = W1 @ X
    assert np.allclose(st.Z, Zp) and np.allclose(Y, W2 @ np.maximum(Zp, 0))
    assert np.allclose(st.G_A, np.maximum(Zp, 0) @ np.maximum(Zp, 0).T)
    assert np.allclose(st.R1, Zp @ X.T) and np.allclose(st.R2, Y @ np.maximum(Zp, 0).T)


def test_first_step_without_pruning_reproduces_pretrained_module():
    # k_keep = n, rho -> 0: the recovered weights reproduce z^pre and y^pre, so a = a^pre and z = z^pre are
    # a fixed point of the loop (the pruning residuals are all zero)
    X, W1, W2 = _small_module(21, d=5, n=8, N=60)
    st, Y = O.ffn_init(X, W1, W2)
    p = O.AdmmParams(rho=1e-12, rho_relative=False, k_keep=8, z_rule="paper")
    Z0 = st.Z.copy()
    s, I, rep, A = O.admm_step(st, X, Y, W1, p)
    assert np.allclose(st.W1, W1, atol=1e-7)
    assert np.allclose(st.W2 @ np.maximum(Z0, 0), Y, atol=1e-7)
    assert np.allclose(A, np.maximum(Z0, 0), atol=1e-7)
    assert np.allclose(st.Z, Z0, atol=1e-7)
    assert rep["res_act"] < 1e-12 and rep["res_out"] < 1e-12 and rep["res_in"] < 1e-12


def test_block_descent_monotone_with_fixed_mask_and_exact_rule():
    X, W1_0, W2_0 = _small_module(22)
    st, Y = O.ffn_init(X, W1_0, W2_0)
    alpha, beta, rho = 1.0, 2.0, 0.05
    p = O.AdmmParams(alpha=alpha, beta=beta, rho=rho, rho_relative=False, k_keep=6, z_rule="exact",
                     reselect_mask=False)
    vals = []
    A = np.maximum(st.Z, 0)
    for it in range(8):
        # objective right after the weight phase, before the auxiliary updates
        O.admm_weight_phase(st, W1_0, p, X.shape[1])
        J_w = O.ffn_objective(st.W1, st.W2, X, Y, st.Z, A, alpha, beta) + alpha * rho * ((st.W1 ** 2).sum() + (st.W2 ** 2).sum())
        Aold, Zold = A, st.Z
        A = O.a_update(st.W2, Y, st.Z, alpha, beta)
        J_a = O.ffn_objective(st.W1, st.W2, X, Y, Zold, A, alpha, beta) + alpha * rho * ((st.W1 ** 2).sum() + (st.W2 ** 2).sum())
        z1, z2 = O.z_candidates(st.W1, X, A, alpha, beta)
        st.Z = O.z_select(Zold, z1, z2, A, alpha, beta, "exact")
        J_z = O.ffn_objective(st.W1, st.W2, X, Y, st.Z, A, alpha, beta) + alpha * rho * ((st.W1 ** 2).sum() + (st.W2 ** 2).sum())
        assert J_a <= J_w * (1 + 1e-12) and J_z <= J_a * (1 + 1e-12)
        if vals:
            assert J_w <= vals[-1] * (1 + 1e-12)      # the weight phase (mask fixed after step 1) does not increase it either
        vals.append(J_z)
        st.G_A = A @ A.T; st.R1 = st.Z @ X.T; st.R2 = Y @ A.T
    assert vals[-1] < vals[0]


def test_pruned_channels_decay_geometrically_while_the_mask_stays():
    """A consequence of the updates of Appendix A.1 that the CUDA path uses to skip work: a pruned channel has a zero
    row in W1 and a zero column in W2, so a = phi(z), z1 = 0 and (ReLU, no dual, either select rule)
    z_new = beta / (alpha + beta) * max(z, 0).  From the second consecutive step with the same mask on, its row of A is
    therefore c = beta / (alpha + beta) times its row of the step before, and so are its row of Z and its columns /
    rows of the accumulators: G_A[pruned, pruned] scales by c^2, R2[:, pruned] and R1[pruned, :] by c.  Checked on the
    oracle's own steps, for both select rules; kept channels do not obey it."""
    X, W1_0, W2_0 = _small_module(31)
    for rule in ("paper", "exact"):
        st, Y = O.ffn_init(X, W1_0, W2_0)
        alpha, beta = 1.3, 0.7
        c = beta / (alpha + beta)
        p = O.AdmmParams(alpha=alpha, beta=beta, rho=0.05, k_keep=5, z_rule=rule)
        prev = None
        obeyed = []
        for it in range(6):
            mask_before = None if st.mask is None else st.mask.copy()
            s, I, rep, A = O.admm_step(st, X, Y, W1_0, p)
            pruned = st.mask == 0
            if prev is not None and np.array_equal(st.mask, prev["mask"]) and prev["mask_before"] is not None \
                    and np.array_equal(prev["mask"], prev["mask_before"]):
                # the same mask in this step, the one before it, and the one before that
                assert np.allclose(A[pruned], c * prev["A"][pruned], rtol=1e-12, atol=0)
                assert np.allclose(st.Z[pruned], c * prev["Z"][pruned], rtol=1e-12, atol=0)
                assert np.allclose(st.G_A[np.ix_(pruned, pruned)], c * c * prev["G_A"][np.ix_(pruned, pruned)], rtol=1e-12)
                assert np.allclose(st.R2[:, pruned], c * prev["R2"][:, pruned], rtol=1e-12)
                assert np.allclose(st.R1[pruned], c * prev["R1"][pruned], rtol=1e-12)
                obeyed.append(it)
            elif prev is not None and np.array_equal(st.mask, prev["mask"]):
                # second step with this mask: A follows already (z of the step before was c max(z, 0) >= 0)
                assert np.allclose(A[pruned], c * prev["A"][pruned], rtol=1e-12, atol=0)
            prev_kept_A = None if prev is None else prev["A"]
            prev = dict(mask=st.mask.copy(), mask_before=mask_before, A=A.copy(), Z=st.Z.copy(), G_A=st.G_A.copy(),
                        R1=st.R1.copy(), R2=st.R2.copy())
        assert obeyed, "the mask never stayed for three steps in this run"
    # the kept channels do not follow the rule
    kept = st.mask == 1
    assert not np.allclose(A[kept], c * prev_kept_A[kept], rtol=1e-3)


def test_admm_step_equals_its_parts_and_keeps_budget():
    X, W1_0, W2_0 = _small_module(23)
    st, Y = O.ffn_init(X, W1_0, W2_0)
    for kind in ("wanda_l2", "wanda_l1", "lemma1"):
        p = O.AdmmParams(k_keep=5, score_kind=kind)
        for _ in range(3):
            s, I, rep, A = O.admm_step(st, X, Y, W1_0, p)
            assert st.mask.sum() == 5                                  # mask budget of Eq. (1)
            assert np.all(st.W1[st.mask == 0] == 0) and np.all(st.W2[:, st.mask == 0] == 0)
            assert np.allclose(st.G_A, A @ A.T) and np.allclose(st.R2, Y @ A.T)
            assert I == pytest.approx(s.mean())


def test_lemma1_in_loop_matches_streamed_definition():
    # the Gram-form used inside the loop (b = W1~ X, c = d = t = z^pre) equals the streamed inner-product form
    X, W1_0, W2_0 = _small_module(24)
    st, Y = O.ffn_init(X, W1_0, W2_0)
    st.R1 = st.R1 + 0.3 * _rng(1).normal(size=st.R1.shape)          # make W1~ differ from W1_0
    p = O.AdmmParams(k_keep=7, score_kind="lemma1", rho=0.2)
    s, I = O.admm_weight_phase(st, W1_0, p, X.shape[1])
    W1t = O.ridge_solve(st.R1, st.G_X, O.effective_ridge(st.G_X, 0.2))
    zpre = W1_0 @ X
    s_ref, rl, _ = O.lemma1_scores(W1t @ X, zpre, zpre, zpre)
    assert np.allclose(s, s_ref, rtol=1e-10)
    assert I == pytest.approx(rl)


def test_dual_mode_drives_primal_residual_down():
    X, W1_0, W2_0 = _small_module(25, d=8, n=10, N=80)
    st, Y = O.ffn_init(X, W1_0, W2_0, dual_mode=True)
    p = O.AdmmParams(alpha=1.0, beta=1.0, rho=0.05, k_keep=6, dual_mode=True, z_rule="exact", reselect_mask=False)
    res = []
    for _ in range(60):
        _, _, rep, _ = O.admm_step(st, X, Y, W1_0, p)
        res.append(rep["res_act"])
    assert res[-1] < 0.05 * max(res[:5])


def test_swiglu_zu_is_stationary_point():
    r = _rng(26)
    a = r.normal(size=50); g = r.normal(size=50); z1 = r.normal(size=50)
    alpha, beta = 0.9, 1.4
    zu = O.swiglu_zu_update(a, g, z1, alpha, beta)
    grad = -2 * beta * g * (a - g * zu) + 2 * alpha * (zu - z1)
    assert np.abs(grad).max() < 1e-12
    assert np.allclose(O.silu(np.array([0.0, 1.0])), [0.0, 1.0 / (1.0 + np.exp(-1.0))])


def test_swiglu_module_special_cases_and_descent():
    """The SwiGLU extension against what the mathematics fixes: with a gate factor of one it is the paper's linear
    branch (z-update = z^(2)), its initial state reproduces the pre-trained module, and with a fixed mask every
    sub-step solves its subproblem exactly, so the FFN objective of Appendix A.1 cannot rise."""
    r = _rng(31)
    d, n, N = 5, 9, 60
    X = r.normal(size=(d, N)); Wg = 0.7 * r.normal(size=(n, d)); Wu = 0.7 * r.normal(size=(n, d))
    W2 = 0.7 * r.normal(size=(d, n))
    # gate factor one: the closed form is z^(2) of "Updating output", duals included
    A = r.normal(size=(n, N)); U = r.normal(size=(n, N)); W1 = r.normal(size=(n, d))
    z1, z2 = O.z_candidates(W1, X, A, 0.8, 1.3, U)
    assert np.allclose(O.swiglu_zu_update(A, np.ones_like(A), z1, 0.8, 1.3, U), z2, atol=1e-13)
    # initial state: the split variables reproduce the module output exactly, token by token
    st, Ypre = O.swiglu_init(X, Wg, Wu, W2)
    for t in (0, 17, N - 1):
        x = X[:, t]
        zg = Wg @ x
        want = W2 @ ((zg / (1.0 + np.exp(-zg))) * (Wu @ x))
        assert np.allclose(Ypre[:, t], want, atol=1e-12)
    assert np.allclose(st.gate * st.Z, O.phi(st.Z, "swiglu", st.gate)) and np.allclose(st.R1, st.Z @ X.T)
    # first step without pruning and a vanishing ridge: the recovered weights are the pre-trained ones, nothing moves
    p = O.AdmmParams(k_keep=n, rho=1e-12, rho_relative=False, act="swiglu")
    st0, _ = O.swiglu_init(X, Wg, Wu, W2)
    _, _, rep, A0 = O.admm_step(st0, X, Ypre, Wu, p)
    assert np.allclose(st0.W1, Wu, atol=1e-6) and np.allclose(st0.W2, W2, atol=1e-6)
    assert rep["res_act"] < 1e-12 and rep["res_in"] < 1e-12 and rep["res_out"] < 1e-12
    # block descent with a fixed mask (the ridge is part of what the recoveries minimise, so keep it negligible)
    p = O.AdmmParams(k_keep=6, rho=1e-10, rho_relative=False, act="swiglu", reselect_mask=True)
    st, _ = O.swiglu_init(X, Wg, Wu, W2)
    prev = None
    for it in range(8):
        _, _, _, A = O.admm_step(st, X, Ypre, Wu, p)
        p.reselect_mask = False
        obj = O.ffn_objective(st.W1, st.W2, X, Ypre, st.Z, A, p.alpha, p.beta, "swiglu", st.gate)
        if prev is not None:
            assert obj <= prev * (1 + 1e-9), (it, obj, prev)
        prev = obj
    assert int(st.mask.sum()) == 6 and np.all(st.W1[st.mask == 0] == 0) and np.all(st.W2[:, st.mask == 0] == 0)
    # stationarity of the a-update with the gated activation
    Ares = O.a_update(st.W2, Ypre, st.Z, 0.9, 1.2, None, "swiglu", st.gate)
    grad = -2 * 0.9 * st.W2.T @ (Ypre - st.W2 @ Ares) + 2 * 1.2 * (Ares - st.gate * st.Z)
    assert np.abs(grad).max() < 1e-9


def test_weight_stats_closed_forms():
    """Algorithm "-distribute" Step 1 statistics against textbook closed forms: the entries 0, 1, ..., m-1 have
    l1 = m(m-1)/2, variance (m^2-1)/12 and sum of squares (m-1)m(2m-1)/6, however they are cut into slices."""
    m = 60
    v = np.arange(m, dtype=np.float64)
    rng = np.random.default_rng(5)
    perm = rng.permutation(m)
    parts = [v[perm[:7]].reshape(7, 1), v[perm[7:31]].reshape(4, 6), v[perm[31:]].reshape(1, 29)]
    l1, var, l2 = O.weight_stats(parts)
    assert l1 == m * (m - 1) / 2
    assert abs(var - (m * m - 1) / 12.0) < 1e-12
    assert abs(l2 - np.sqrt((m - 1) * m * (2 * m - 1) / 6.0)) < 1e-12
    # signs: the l1 norm ignores them, the variance does not (a +-1 checkerboard has mean 0, variance 1)
    cb = np.where((np.add.outer(np.arange(6), np.arange(8)) % 2) == 0, 1.0, -1.0)
    assert O.weight_stats([cb]) == (48.0, 1.0, np.sqrt(48.0))
    assert O.weight_stats([np.full((3, 5), -2.0)]) == (30.0, 0.0, np.sqrt(60.0))
    # scaling by c: l1 and l2 scale with |c|, the variance with c^2
    a = rng.standard_normal((5, 9))
    s1, s3 = O.weight_stats([a]), O.weight_stats([-3.0 * a])
    assert abs(s3[0] - 3 * s1[0]) < 1e-12 and abs(s3[1] - 9 * s1[1]) < 1e-12 and abs(s3[2] - 3 * s1[2]) < 1e-12


def test_distribute_importance_structure():
    """Depth decay, the attention/MLP ratio and the head slicing of Algorithm "-distribute" Step 1."""
    d, n, H = 8, 12, 4
    dh = d // H
    rng = np.random.default_rng(9)
    base = dict(Wq=rng.standard_normal((d, d)), Wk=rng.standard_normal((d, d)), Wv=rng.standard_normal((d, d)),
                Wo=rng.standard_normal((d, d)), fc1=rng.standard_normal((n, d)), fc2=rng.standard_normal((d, n)))
    layers = [base, base, base]
    Ia, Im = O.distribute_importance(layers, H, dh, rho=2.5, gamma=0.9)
    # identical layers: consecutive importances differ by the factor gamma; layer 1 carries gamma^1
    assert np.allclose(Ia[1:] / Ia[:-1], 0.9) and np.allclose(Im[1:] / Im[:-1], 0.9)
    Ia1, Im1 = O.distribute_importance(layers, H, dh, rho=1.0, gamma=1.0)
    assert np.allclose(Ia, 2.5 * Ia1 * 0.9 ** np.arange(1, 4)) and np.allclose(Im, Im1 * 0.9 ** np.arange(1, 4))
    # the MLP term by hand: l1 and population variance of fc1 and fc2
    want = sum(np.abs(base[k]).sum() + 0.05 * base[k].var() for k in ("fc1", "fc2"))
    assert abs(Im1[0] - want) < 1e-9 * want
    # head slicing: the l1 parts of all heads together are the l1 norms of the four attention matrices
    l1_heads = sum(O.weight_stats(O.head_slices(base["Wq"], base["Wk"], base["Wv"], base["Wo"], h, dh))[0]
                   for h in range(H))
    assert abs(l1_heads - sum(np.abs(base[k]).sum() for k in ("Wq", "Wk", "Wv", "Wo"))) < 1e-9
    # a head whose weights are zero contributes nothing; only W_O's COLUMNS of that head count
    z = {k: v.copy() for k, v in base.items()}
    z["Wq"][:dh] = 0; z["Wk"][:dh] = 0; z["Wv"][:dh] = 0; z["Wo"][:, :dh] = 0
    parts0 = O.head_slices(z["Wq"], z["Wk"], z["Wv"], z["Wo"], 0, dh)
    assert O.weight_stats(parts0) == (0.0, 0.0, 0.0)
    z["Wo"][:dh, dh:] = 7.0      # rows of W_O are not part of head 0
    assert O.weight_stats(O.head_slices(z["Wq"], z["Wk"], z["Wv"], z["Wo"], 0, dh)) == (0.0, 0.0, 0.0)
    # inverse allocation on these importances, as printed (Step 2): w falls with the importance, r = rbar L (1 - w) /
    # sum(1 - w) rises with it, so the first (most important, least decayed) layer gets the largest pruned fraction;
    # the mean stays rbar
    r, _ = O.allocate_sparsity(Im, np.full(3, n), 0.5, T=float(np.abs(Im).mean()), mode="inverse")
    assert np.all(np.diff(Im) < 0) and np.all(np.diff(r) < 0) and abs(r.mean() - 0.5) < 1e-12


def _frac(tok):
    num, _, den = tok.partition("/")
    return float(num) / float(den) if den else float(num)


def test_distribute_importance_golden():
    """Algorithm "-distribute", Step 1 on hand-evaluated 2 x 2 weights (tests/golden/distribute_cases.txt): pins the
    coefficients 0.1 (variance) and 0.01 (l2 norm) of the head term, 0.05 of the MLP term, the head slicing, the
    attention/MLP ratio and the depth weight gamma^l with layers counted from 1."""
    rows = {}
    for ln in _rows("distribute_cases.txt"):
        name, vals = ln.split("|")
        rows[name.strip()] = [float(v) for v in vals.split()]
    layer = {k: np.array(rows[k]).reshape(2, 2) for k in ("Wq", "Wk", "Wv", "Wo", "fc1", "fc2")}
    rho, gamma = rows["rho_gamma"]
    for h, want in enumerate(rows["head_terms"]):
        l1, var, l2 = O.weight_stats(O.head_slices(layer["Wq"], layer["Wk"], layer["Wv"], layer["Wo"], h, 1))
        assert l1 + 0.1 * var + 0.01 * l2 == pytest.approx(want, rel=1e-13)
    Ia, Im = O.distribute_importance([layer, layer], 2, 1, rho=rho, gamma=gamma)
    assert np.allclose(Ia, rows["I_attn"], rtol=1e-13, atol=0)
    assert np.allclose(Im, rows["I_mlp"], rtol=1e-13, atol=0)


def test_inverse_allocation_golden():
    """Algorithm "-distribute", Step 2 with rational softmax weights, one case without and one with the clip."""
    T = 0.83
    for ln in _rows("inverse_allocation_cases.txt"):
        rbar_s, n_s, q_s, r_s, k_s = ln.split("|")
        q = np.array([_frac(t) for t in q_s.split()])
        want_r = np.array([_frac(t) for t in r_s.split()])
        want_k = [int(t) for t in k_s.split()]
        I = -T * np.log(q)
        r, k = O.allocate_sparsity(I, [int(n_s)] * len(q), float(rbar_s), T, mode="inverse")
        assert np.allclose(r, want_r, rtol=1e-12, atol=0)
        assert list(k) == want_k


# ------------------------------------------------------------------------------------------------ global threshold
def test_global_threshold_worked_example():
    """Appendix B, Algorithm 3: one threshold over the scores of all layers, K = floor(r n L) kept.  Two layers of three
    units, half kept: the three largest of {5, 1, 3, 4, 2, 6} are 6, 5, 4 — one unit of layer 0, two of layer 1."""
    S = np.array([[5.0, 1.0, 3.0], [4.0, 2.0, 6.0]])
    masks, counts, tau = O.global_threshold_masks(S, 0.5)
    assert masks.tolist() == [[1, 0, 0], [1, 0, 1]] and counts.tolist() == [1, 2] and tau == 4.0
    # K = floor(r n L): 0.6 * 6 = 3.6 -> 3 as well; 2/3 -> 4 kept
    assert O.global_threshold_masks(S, 0.6)[1].sum() == 3
    assert O.global_threshold_masks(S, 2.0 / 3.0)[0].tolist() == [[1, 0, 1], [1, 0, 1]]


def test_global_threshold_properties_and_special_cases():
    rng = np.random.default_rng(5)
    for L, n, r in ((1, 40, 0.3), (4, 33, 0.5), (7, 20, 0.85)):
        S = np.round(rng.normal(size=(L, n)) * 4) / 4            # many exact ties, also across layers
        masks, counts, tau = O.global_threshold_masks(S, r)
        K = int(np.floor(r * n * L + 1e-9))
        assert masks.sum() == K == counts.sum()
        kept, pruned = S[masks == 1], S[masks == 0]
        assert kept.min() >= pruned.max() and kept.min() == tau    # a single threshold separates the two sets
        # ties at the threshold: the kept ones come first in (layer, index) order
        at = np.flatnonzero(S.reshape(-1) == tau)
        m_at = masks.reshape(-1)[at]
        assert np.all(np.diff(m_at.astype(int)) <= 0)
        # brute force: repeatedly take the largest remaining score, earliest position first
        flat = S.reshape(-1).copy()
        ref = np.zeros(L * n, np.uint8)
        for _ in range(K):
            j = int(np.argmax(flat))                                # argmax returns the first maximum
            ref[j] = 1
            flat[j] = -np.inf
        assert np.array_equal(ref.reshape(L, n), masks)
        if L == 1:                                                  # one layer: the per-layer top-k of Algorithm 1
            assert np.array_equal(masks[0], O.topk_mask(S[0], K)[0])
    # equal score distributions in every layer -> the global threshold is the uniform allocation
    base = rng.permutation(50).astype(float)
    S = np.stack([rng.permutation(base) for _ in range(5)])
    assert O.global_threshold_masks(S, 0.4)[1].tolist() == [20] * 5


def test_global_threshold_can_empty_a_layer_unless_min_keep():
    S = np.array([[9.0, 8.0, 7.0], [1.0, 2.0, 3.0]])
    masks, counts, _ = O.global_threshold_masks(S, 0.5)
    assert counts.tolist() == [3, 0]
    masks, counts, _ = O.global_threshold_masks(S, 0.5, min_keep=1)
    assert masks.tolist() == [[1, 1, 1], [0, 0, 1]] and counts.tolist() == [3, 1]


# ------------------------------------------------------------------------------------------------ Algorithm 1, one temperature
def test_temperature_loss_special_cases():
    """L(T) of Algorithm 1 Step 5 against what the paper's construction fixes: with nothing pruned (rbar = 0) and a
    vanishing ridge the recovered weights are the pre-trained ones and every term of the objective is zero, at any
    temperature; identical layers get the uniform allocation, so L(T) is L times one layer's loss for every T; and the
    kept counts follow Step 2 (softmax of -I/T at T = T_rel mean|I|: the least important layer is pruned most)."""
    rng = _rng(31)
    d, n, N = 6, 14, 60
    mk = lambda s: (rng.standard_normal((d, N)), s * rng.standard_normal((n, d)), rng.standard_normal((d, n)))
    layers = [mk(1.0), mk(2.0), mk(3.0)]
    p = O.AdmmParams(rho=1e-10, rho_relative=False)
    for T_rel in (0.3, 3.0):
        L0, per, r, k = O.temperature_loss(layers, 0.0, T_rel, 2, p)
        scale = sum(np.linalg.norm(W2 @ np.maximum(W1 @ X, 0)) ** 2 for X, W1, W2 in layers)
        assert np.all(r == 0) and list(k) == [n] * 3 and L0 < 1e-12 * scale
    same = [layers[1]] * 3
    La, per_a, r_a, k_a = O.temperature_loss(same, 0.5, 0.3, 2, O.AdmmParams(rho=0.1))
    Lb, per_b, r_b, k_b = O.temperature_loss(same, 0.5, 3.0, 2, O.AdmmParams(rho=0.1))
    assert np.allclose(r_a, 0.5) and np.allclose(r_b, 0.5) and list(k_a) == [7] * 3
    assert La == pytest.approx(3 * per_a[0], rel=1e-12) and La == pytest.approx(Lb, rel=1e-12) and La > 0
    # different layers: importances grow with the weight scale, so the first layer is pruned most, and the lower the
    # temperature the more uneven the kept counts
    _, _, r_lo, k_lo = O.temperature_loss(layers, 0.5, 0.3, 1, O.AdmmParams(rho=0.1))
    _, _, r_hi, k_hi = O.temperature_loss(layers, 0.5, 3.0, 1, O.AdmmParams(rho=0.1))
    assert np.all(np.diff(r_lo) < 0) and np.all(np.diff(r_hi) < 0)
    assert (k_lo.max() - k_lo.min()) > (k_hi.max() - k_hi.min())
