"""CPU fp64 oracle for the per-module ADMM path of structured SparseLLM / STRUPRUNE.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the paper computes.  It
shares no code with the CUDA library and must never be imported by the product path; only the tests,
the smoke check and the benchmark's CPU-baseline leg may call it.

Conventions follow the paper: a calibration tensor holds one token per COLUMN, so the module input
is X = a_{l-1}^pre in R^{d x N}, the up-projection is W1 = W_l in R^{n x d}, the down-projection is
W2 = W_{l+1} in R^{d x n}, the auxiliary variables are Z = z_l and A = a_l in R^{n x N}, and the
pre-trained module output is Ypre = z_{l+1}^pre in R^{d x N}.  (The CUDA library stores the same
tensors token-major, i.e. the transposes.)  Everything is float64 numpy.

Readings of points where the paper is silent or inconsistent (each is a named switch here and is
implemented identically by the CUDA path):
  * ridge: the weight recovery W = z a^+ (Appendix A.1, "Reversely recovering the weight matrix") is
    computed as the Tikhonov-regularised least squares W = R (G + rho_eff I)^-1 with G = a a^T and
    R = z a^T.  rho_eff = rho * trace(G)/dim(G) when `rho_relative`, else rho.  rho -> 0 with a of
    full row rank gives z a^+ back.
  * a-update: the formula of Appendix A.1 ("Updating activation") and Algorithm 3 (GSPO), not the
    dimensionally inconsistent copy printed in Algorithm 2.
  * z-update: rule "paper" is the literal select of Algorithms 2 and 3 (test the OLD z, strict < 0);
    rule "exact" is the true minimiser of the scalar problem in "Updating output".
  * dual variables: absent from the paper.  dual_mode adds the textbook scaled dual U of the
    constraint a = phi(z): phi(z) is replaced by phi(z) - U in the a-update, a by a + U in the
    z-update, and U += a - phi(z) afterwards.  U = 0 reproduces the paper exactly.
  * Lemma 1 over N calibration tokens: products of scalars become inner products over tokens.
  * threshold: exactly k units are kept (the k largest scores, lower index wins ties, NaN lowest), so
    that the mask budget of Eq. (1) holds with equality.
  * "-distribute" importances: a head's weight matrix W_h is read as its rows of W_Q, W_K, W_V and its
    columns of W_O taken together; Var is the population variance over those entries; layers count from 1.
  * allocation: r_l is the fraction PRUNED in layer l, as Algorithm 1 uses it (clip at 0.95, "mask with
    sparsity r_l"); kept count = n_l - round_half_up(r_l n_l).

Pins.  Every function is pinned by tests/test_oracle_pins.py and tests/test_oracle_mha_pins.py to
something other than itself: values the paper's formulas give by hand (golden files), closed forms,
stationarity and finite-difference checks, brute force on tiny inputs, special cases that reduce to a
library routine.  Two groups have no printed number or worked example in the paper to compare with, so
their pins are mathematical only and the READING they implement is a choice stated above them: the
SwiGLU extension (`swiglu_init`, `swiglu_zu_update`, the gated branches) and the multi-head attention
functions `mha_*` (Method 2 is printed with inconsistent shapes and without step sizes).
Parity unpinned: the default values of alpha, beta, rho, T (the paper fixes none of them).
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------------------------------
# Gram and cross products (what W = z a^+ needs; Appendix A.1 "Reversely recovering the weight matrix")
# --------------------------------------------------------------------------------------------------
def gram_accumulate(G, R, Xc, Yc=None, rowstats=None):
    """G += Xc Xc^T, R += Yc Xc^T over one chunk of token columns; rowstats[:,0] += sum|x|, [:,1] += sum x^2."""
    Xc = np.asarray(Xc, F64)
    G += Xc @ Xc.T
    if Yc is not None:
        R += np.asarray(Yc, F64) @ Xc.T
    if rowstats is not None:
        rowstats[:, 0] += np.abs(Xc).sum(axis=1)
        rowstats[:, 1] += (Xc * Xc).sum(axis=1)
    return G, R


def effective_ridge(G, rho, rho_relative=True):
    """rho_eff of the Tikhonov term (see header)."""
    G = np.asarray(G, F64)
    return float(rho) * float(np.trace(G)) / G.shape[0] if rho_relative else float(rho)


def ridge_solve(R, G, rho_eff):
    """W = R (G + rho_eff I)^-1  — regularised form of W = z a^+ (Appendix A.1)."""
    G = np.asarray(G, F64)
    K = G + rho_eff * np.eye(G.shape[0])
    return np.linalg.solve(K, np.asarray(R, F64).T).T  # K symmetric


def restricted_refit(R, G, keep, rho_eff):
    """Recovery solver on a kept support S (Algorithm 2, "prune by importance + recovery solver"):
    W[:, S] = R[:, S] (G[S,S] + rho_eff I)^-1, W[:, S^c] = 0."""
    R = np.asarray(R, F64)
    G = np.asarray(G, F64)
    S = np.flatnonzero(np.asarray(keep))
    W = np.zeros_like(R)
    if S.size:
        W[:, S] = ridge_solve(R[:, S], G[np.ix_(S, S)], rho_eff)
    return W


# --------------------------------------------------------------------------------------------------
# Activation, a-update, z-update (Appendix A.1; Algorithm 3 lines for a_l, z^(1), z^(2), select)
# --------------------------------------------------------------------------------------------------
def phi(Z, act="relu", gate=None):
    """Activation of the module: ReLU (the paper's case), or the gated form g * z of the SwiGLU extension, where
    g = SiLU(gate pre-activation) is a fixed factor per entry (see the SwiGLU section below)."""
    Z = np.asarray(Z, F64)
    if act == "relu":
        return np.maximum(Z, 0.0)
    if act == "swiglu":
        return np.asarray(gate, F64) * Z
    raise ValueError(act)


def a_update(W2, Ypre, Z, alpha, beta, U=None, act="relu", gate=None):
    """a_l = (alpha W2^T W2 + beta I)^-1 (alpha W2^T Ypre + beta (phi(z_l) - U))."""
    W2 = np.asarray(W2, F64)
    n = W2.shape[1]
    H = phi(Z, act, gate) - (0.0 if U is None else np.asarray(U, F64))
    lhs = alpha * (W2.T @ W2) + beta * np.eye(n)
    rhs = alpha * (W2.T @ np.asarray(Ypre, F64)) + beta * H
    return np.linalg.solve(lhs, rhs)


def z_candidates(W1, X, A, alpha, beta, U=None):
    """z^(1) = W1 X and z^(2) = (beta (a + U) + alpha z^(1)) / (alpha + beta)."""
    z1 = np.asarray(W1, F64) @ np.asarray(X, F64)
    Au = np.asarray(A, F64) + (0.0 if U is None else np.asarray(U, F64))
    z2 = (beta * Au + alpha * z1) / (alpha + beta)
    return z1, z2


def z_exact_candidates(z1, z2, A, alpha, beta, U=None):
    """Best point of each half line of the scalar problem beta (a - relu(z))^2 + alpha (z - z1)^2 and its value:
    returns (zn, zp, fn, fp) with zn = min(z1, 0) on z <= 0 and zp = max(z2, 0) on z >= 0."""
    Au = np.asarray(A, F64) + (0.0 if U is None else np.asarray(U, F64))
    zn = np.minimum(z1, 0.0)
    zp = np.maximum(z2, 0.0)
    fn = beta * Au ** 2 + alpha * (zn - z1) ** 2
    fp = beta * (Au - zp) ** 2 + alpha * (zp - z1) ** 2
    return zn, zp, fn, fp


def z_select(Zold, z1, z2, A, alpha, beta, rule="paper", U=None):
    """Elementwise select of the z-update."""
    Zold = np.asarray(Zold, F64)
    if rule == "paper":
        # Algorithms 2/3: entry takes z^(1) if the current z entry is negative, z^(2) otherwise.
        return np.where(Zold < 0.0, z1, z2)
    if rule == "exact":
        # argmin_z beta (a - relu(z))^2 + alpha (z - z1)^2: best point of each half line, then compare.
        zn, zp, fn, fp = z_exact_candidates(z1, z2, A, alpha, beta, U)
        return np.where(fn < fp, zn, zp)
    raise ValueError(rule)


def dual_update(U, A, Znew, act="relu", gate=None):
    """Scaled dual ascent on a = phi(z) (not in the paper; see header)."""
    return np.asarray(U, F64) + np.asarray(A, F64) - phi(Znew, act, gate)


# --------------------------------------------------------------------------------------------------
# Structured scores (Lemma 1 / Eq. (3); Section 3.4 Eq. (Wanda); Algorithm 1 Step 3)
# --------------------------------------------------------------------------------------------------
def _group_sum(v, group):
    v = np.asarray(v, F64)
    assert v.shape[0] % group == 0
    return v.reshape(v.shape[0] // group, group).sum(axis=1)


def lemma1_scores(b, c, dd, t, group=1):
    """s_j = (<c_j,b_j> + <d_j,t_j>) / (|c_j|^2 + |d_j|^2) with inner products over tokens (columns);
    t is the target paired with d (printed z^pre in Lemma 1).  With N = 1 this is Eq. (3) literally.
    A unit made of `group` consecutive rows sums numerators and denominators over its rows.
    Returns (scores, layer value r_l = mean_j s_j (Lemma 1, derivation form 1/n sum over units), e_j)."""
    b, c, dd, t = (np.asarray(v, F64).reshape(np.shape(v)[0], -1) for v in (b, c, dd, t))
    num = _group_sum((c * b).sum(axis=1) + (dd * t).sum(axis=1), group)
    den = _group_sum((c * c).sum(axis=1) + (dd * dd).sum(axis=1), group)
    s = num / den
    return s, float(s.mean()), den


def relaxed_mask(s, e, r_layer):
    """Relaxed mask of Appendix B (Eq. Mlj): M_j = s_j - (1/e_j) (sum_k s_k - r_l n) / sum_k (1/e_k)."""
    s = np.asarray(s, F64)
    e = np.asarray(e, F64)
    n = s.shape[0]
    lam_half = (s.sum() - r_layer * n) / (1.0 / e).sum()
    return s - lam_half / e


def wanda_scores(W, colsq=None, colabs_mean=None, kind="l2", group=1):
    """Structured Wanda score of the units feeding the columns of W (W in R^{out x n}).
    l2 (Eq. Wanda): elementwise |W_ij| * |a_j|_2 reduced with the l2 norm over the unit's block,
        i.e. sqrt(sum_{j in unit} |W[:,j]|_2^2 * colsq_j), colsq_j = sum_t a_jt^2.
    l1 (Algorithm 1, Step 3): sum_{j in unit} |W[:,j]|_1 * mean_t |a_jt|.
    Returns (scores, layer importance I = mean over units)."""
    W = np.asarray(W, F64)
    if kind == "l2":
        per = (W * W).sum(axis=0) * np.asarray(colsq, F64)
        s = np.sqrt(_group_sum(per, group))
    elif kind == "l1":
        per = np.abs(W).sum(axis=0) * np.asarray(colabs_mean, F64)
        s = _group_sum(per, group)
    else:
        raise ValueError(kind)
    return s, float(s.mean())


# --------------------------------------------------------------------------------------------------
# Softmax allocation (Lemma 2; Algorithm 1 Step 2; Algorithm 2' inverse weighting)
# --------------------------------------------------------------------------------------------------
def _round_half_up(x):
    return int(math.floor(x + 0.5))


def allocate_sparsity(I, n_units, rbar, T, mode="softmax", clip_hi=0.95):
    """Per-layer pruned fractions r_l and kept counts.
    softmax: w = softmax(-I/T); r = rbar L w; clip to [0, clip_hi]; if nothing hit clip_hi, rescale to mean
             rbar and clip again (Algorithm 1, Step 2).
    inverse: r = clip(rbar L (1 - w)/sum(1 - w), 0, clip_hi)      (Algorithm "-distribute", Step 2).
    uniform: r = rbar."""
    I = np.asarray(I, F64)
    L = I.shape[0]
    if mode == "uniform":
        r = np.full(L, float(rbar))
    else:
        a = -I / T
        a = a - a.max()
        w = np.exp(a)
        w = w / w.sum()
        if mode == "softmax":
            raw = rbar * L * w
            r = np.minimum(np.maximum(raw, 0.0), clip_hi)
            if not np.any(raw > clip_hi):
                mu = r.mean()
                if mu > 0:
                    r = r * (rbar / mu)
                r = np.minimum(np.maximum(r, 0.0), clip_hi)
        elif mode == "inverse":
            r = rbar * L * (1.0 - w) / (1.0 - w).sum() if L > 1 else np.full(L, float(rbar))
            r = np.minimum(np.maximum(r, 0.0), clip_hi)
        else:
            raise ValueError(mode)
    n_units = np.asarray(n_units, np.int64)
    k_keep = np.array([int(n_units[l]) - _round_half_up(r[l] * int(n_units[l])) for l in range(L)], np.int64)
    return r, k_keep


# --------------------------------------------------------------------------------------------------
# Weight-statistic importances (Algorithm "-distribute", Step 1)
# --------------------------------------------------------------------------------------------------
def weight_stats(parts):
    """(l1 norm, variance, l2 norm) of the entries of one or several weight slices taken together
    (Algorithm "-distribute", Step 1: the three statistics of a head's or a layer's weight matrix).
    The variance is the population variance over all entries; the l2 norm is the root of the sum of squares."""
    v = np.concatenate([np.asarray(p, F64).ravel() for p in parts])
    m = v.shape[0]
    mean = v.sum() / m
    return float(np.abs(v).sum()), float(((v - mean) ** 2).sum() / m), float(math.sqrt((v * v).sum()))


def head_slices(Wq, Wk, Wv, Wo, h, d_head):
    """The weights of attention head h: its d_head rows of W_Q, W_K, W_V and its d_head columns of W_O."""
    r = slice(h * d_head, (h + 1) * d_head)
    return [np.asarray(Wq)[r, :], np.asarray(Wk)[r, :], np.asarray(Wv)[r, :], np.asarray(Wo)[:, r]]


def distribute_importance(layers, n_heads, d_head, rho, gamma):
    """Algorithm "-distribute", Step 1.  layers[l] = dict(Wq, Wk, Wv, Wo, fc1, fc2); layer l (counted from 1 as
    the algorithm does) has depth weight d_l = gamma^l.
      I_attn[l] = d_l rho sum_h (|W_h|_1 + 0.1 Var(W_h) + 0.01 |W_h|_2)
      I_mlp[l]  = d_l sum_{m in fc1, fc2} (|W_m|_1 + 0.05 Var(W_m))"""
    L = len(layers)
    I_attn, I_mlp = np.zeros(L, F64), np.zeros(L, F64)
    for l, w in enumerate(layers):
        dl = gamma ** (l + 1)
        acc = 0.0
        for h in range(n_heads):
            l1, var, l2 = weight_stats(head_slices(w["Wq"], w["Wk"], w["Wv"], w["Wo"], h, d_head))
            acc += l1 + 0.1 * var + 0.01 * l2
        I_attn[l] = dl * rho * acc
        acc = 0.0
        for name in ("fc1", "fc2"):
            l1, var, _ = weight_stats([w[name]])
            acc += l1 + 0.05 * var
        I_mlp[l] = dl * acc
    return I_attn, I_mlp


# --------------------------------------------------------------------------------------------------
# Top-k mask and mask application (Algorithm 1 Step 3; Algorithm 3 threshold + M (.) W)
# --------------------------------------------------------------------------------------------------
def topk_mask(scores, k_keep):
    """Keep exactly the k largest scores (ties: lower index kept; NaN sorts lowest).  Returns (mask u8, tau)."""
    s = np.asarray(scores, F64).copy()
    n = s.shape[0]
    s[np.isnan(s)] = -np.inf
    order = np.lexsort((np.arange(n), -s))  # primary: descending score, secondary: ascending index
    mask = np.zeros(n, np.uint8)
    k = int(k_keep)
    if k > 0:
        mask[order[:k]] = 1
    tau = float(s[order[k - 1]]) if 0 < k <= n else float("nan")
    return mask, tau


def global_threshold_masks(scores_per_layer, keep_fraction, min_keep=0):
    """Appendix B, Algorithm 3 (GSPO), threshold step: the scores of all L layers are collected, K = floor(r n L)
    with r the kept fraction of the global budget, and the units holding the K largest scores are kept — one
    threshold for the whole model, so layers end with different kept counts.  Exactly K units are kept (ties: the
    earlier layer, then the lower index).  min_keep > 0: a layer left with fewer units keeps its own min_keep
    largest instead (the algorithm as printed can empty a layer).  Returns (masks u8 [L, n], kept counts, tau)."""
    S = np.asarray(scores_per_layer, F64)
    L, n = S.shape
    K = int(np.floor(keep_fraction * n * L + 1e-9))
    flat, tau = topk_mask(S.reshape(-1), K)
    masks = flat.reshape(L, n).copy()
    for l in range(L):
        if masks[l].sum() < min_keep:
            masks[l], _ = topk_mask(S[l], min_keep)
    return masks, masks.sum(axis=1).astype(np.int64), tau


def apply_mask(mask, group=1, W_rows=None, W_cols=None):
    """M (.) W: zero the row groups of W_rows and the column groups of W_cols of pruned units."""
    m = np.repeat(np.asarray(mask).astype(bool), group)
    out_r = None if W_rows is None else np.where(m[:, None], np.asarray(W_rows, F64), 0.0)
    out_c = None if W_cols is None else np.where(m[None, :], np.asarray(W_cols, F64), 0.0)
    return out_r, out_c


# --------------------------------------------------------------------------------------------------
# The FFN module loop (Algorithm 2, SparseLLM1, merged with Algorithm 3's per-step order)
# --------------------------------------------------------------------------------------------------
@dataclasses.dataclass
class AdmmParams:
    alpha: float = 1.0
    beta: float = 1.0
    rho: float = 0.1
    rho_relative: bool = True
    z_rule: str = "paper"
    dual_mode: bool = False
    score_kind: str = "wanda_l2"  # "wanda_l2" | "wanda_l1" | "lemma1"
    k_keep: int = 0
    reselect_mask: bool = True
    refit: bool = True
    act: str = "relu"


@dataclasses.dataclass
class FfnState:
    Z: np.ndarray
    U: np.ndarray | None
    G_X: np.ndarray
    G_A: np.ndarray
    R1: np.ndarray
    R2: np.ndarray
    absA: np.ndarray  # sum_t |a_jt| of the A that produced G_A
    W1: np.ndarray | None = None
    W2: np.ndarray | None = None
    mask: np.ndarray | None = None
    it: int = 0
    gate: np.ndarray | None = None   # SwiGLU extension: g = SiLU(Wg X), fixed over the iterations


def ffn_init(X, W1_0, W2_0, act="relu", dual_mode=False):
    """Initialisation of SparseLLM1: z = z^pre = W1_0 X, a = a^pre = phi(z^pre), target Ypre = W2_0 a^pre,
    and the Gram / cross products the first weight recovery needs."""
    X = np.asarray(X, F64)
    Zpre = np.asarray(W1_0, F64) @ X
    Apre = phi(Zpre, act)
    Ypre = np.asarray(W2_0, F64) @ Apre
    st = FfnState(
        Z=Zpre.copy(), U=np.zeros_like(Zpre) if dual_mode else None,
        G_X=X @ X.T, G_A=Apre @ Apre.T, R1=Zpre @ X.T, R2=Ypre @ Apre.T, absA=np.abs(Apre).sum(axis=1))
    return st, Ypre


def admm_weight_phase(st, W1_0, p, N):
    """Weight recovery, unit scores, top-k mask and recovery on the kept support for the current accumulators."""
    rho1 = effective_ridge(st.G_X, p.rho, p.rho_relative)
    rho2 = effective_ridge(st.G_A, p.rho, p.rho_relative)
    W1t = ridge_solve(st.R1, st.G_X, rho1)          # W_l     = z_l a_{l-1}^+
    W2t = ridge_solve(st.R2, st.G_A, rho2)          # W_{l+1} = z_{l+1}^pre a_l^+
    if p.score_kind == "wanda_l2":
        s, I = wanda_scores(W2t, colsq=np.diag(st.G_A), kind="l2")
    elif p.score_kind == "wanda_l1":
        s, I = wanda_scores(W2t, colabs_mean=st.absA / N, kind="l1")
    elif p.score_kind == "lemma1":
        # b = W1~ X, c = d = t = z^pre = W1_0 X, all expressed through G_X = X X^T
        W10 = np.asarray(W1_0, F64)
        cb = ((W10 @ st.G_X) * W1t).sum(axis=1)
        cc = ((W10 @ st.G_X) * W10).sum(axis=1)
        s = (cb + cc) / (2.0 * cc)
        I = float(s.mean())
    else:
        raise ValueError(p.score_kind)
    if p.reselect_mask or st.mask is None:
        st.mask, tau = topk_mask(s, p.k_keep)
    W1, _ = apply_mask(st.mask, 1, W_rows=W1t)       # row masking is already the restricted solution for W1
    if p.refit:
        W2 = restricted_refit(st.R2, st.G_A, st.mask, rho2)
    else:
        _, W2 = apply_mask(st.mask, 1, W_cols=W2t)
    st.W1, st.W2 = W1, W2
    return s, I


def admm_step(st, X, Ypre, W1_0, p):
    """One outer step: weights from the accumulators, then a-, z- (and dual) updates, then the accumulators
    of the new auxiliary variables.  Returns (scores, layer importance, report dict, A)."""
    X = np.asarray(X, F64)
    Ypre = np.asarray(Ypre, F64)
    N = X.shape[1]
    s, I = admm_weight_phase(st, W1_0, p, N)
    U = st.U if p.dual_mode else None
    A = a_update(st.W2, Ypre, st.Z, p.alpha, p.beta, U, p.act, st.gate)
    z1, z2 = z_candidates(st.W1, X, A, p.alpha, p.beta, U)
    if p.act == "swiglu":
        Znew = swiglu_zu_update(A, st.gate, z1, p.alpha, p.beta, U)    # one closed form, no select
    else:
        Znew = z_select(st.Z, z1, z2, A, p.alpha, p.beta, p.z_rule, U)
    if p.dual_mode:
        st.U = dual_update(st.U, A, Znew, p.act, st.gate)
    st.Z = Znew
    st.G_A = A @ A.T
    st.R1 = Znew @ X.T
    st.R2 = Ypre @ A.T
    st.absA = np.abs(A).sum(axis=1)
    st.it += 1
    rep = {
        "res_act": float(((A - phi(Znew, p.act, st.gate)) ** 2).sum()),
        "res_out": float(p.alpha * ((Ypre - st.W2 @ A) ** 2).sum()),
        "res_in": float(p.alpha * ((Znew - st.W1 @ X) ** 2).sum()),
    }
    return s, I, rep, A


def ffn_objective(st_W1, st_W2, X, Ypre, Z, A, alpha, beta, act="relu", gate=None):
    """alpha |Ypre - W2 A|^2 + beta |A - phi(Z)|^2 + alpha |Z - W1 X|^2 (Appendix A.1, FFN objective)."""
    X = np.asarray(X, F64)
    return (alpha * ((np.asarray(Ypre, F64) - st_W2 @ A) ** 2).sum()
            + beta * ((A - phi(Z, act, gate)) ** 2).sum()
            + alpha * ((Z - st_W1 @ X) ** 2).sum())


# --------------------------------------------------------------------------------------------------
# Algorithm 1 for one temperature: Steps 1-5 over the FFN modules of a model, L(T) = sum_l L_l
# --------------------------------------------------------------------------------------------------
def pretrained_importance(X, W1_0, W2_0, kind="wanda_l2"):
    """Step 1 of Algorithm 1 for one FFN module: I_l = mean unit score of the pre-trained down-projection against the
    pre-trained activation a^pre = phi(W1_0 X) (the Wanda score of Section 3.4 / Step 3 on the unpruned module)."""
    A = phi(np.asarray(W1_0, F64) @ np.asarray(X, F64))
    if kind == "wanda_l2":
        return wanda_scores(W2_0, colsq=(A * A).sum(axis=1), kind="l2")[1]
    if kind == "wanda_l1":
        return wanda_scores(W2_0, colabs_mean=np.abs(A).mean(axis=1), kind="l1")[1]
    raise ValueError(kind)


def temperature_loss(layers, rbar, T_rel, iters, p, mode="softmax"):
    """Algorithm 1 for ONE temperature of its grid.  layers[l] = (X, W1_0, W2_0) of FFN module l (tokens are columns).
      Step 1  I_l of every pre-trained module
      Step 2  r_l from the softmax allocation at temperature T = T_rel * mean_l |I_l| (the temperature is given
              relative to the magnitude of the importances), kept count per layer
      Step 3/4  the module iterations of Algorithm 2 with that kept count (at least one unit)
      Step 5  L(T) = sum_l L_l with L_l the FFN objective of Appendix A.1 after the last iteration
    Returns (L(T), per-layer losses, r, kept counts)."""
    L = len(layers)
    I = np.array([pretrained_importance(X, W1, W2, p.score_kind) for (X, W1, W2) in layers], F64)
    T = T_rel * float(np.abs(I).mean())
    n_units = [np.shape(W1)[0] for (_, W1, _) in layers]
    r, k_keep = allocate_sparsity(I, n_units, rbar, T, mode)
    losses = np.zeros(L, F64)
    for l, (X, W1_0, W2_0) in enumerate(layers):
        st, Ypre = ffn_init(X, W1_0, W2_0, dual_mode=p.dual_mode)
        pl = dataclasses.replace(p, k_keep=max(1, int(k_keep[l])))
        A = None
        for _ in range(iters):
            _, _, _, A = admm_step(st, X, Ypre, W1_0, pl)
        losses[l] = ffn_objective(st.W1, st.W2, X, Ypre, st.Z, A, p.alpha, p.beta)
    return float(losses.sum()), losses, r, k_keep


# --------------------------------------------------------------------------------------------------
# SwiGLU extension (not in the paper: its modules are ReLU FFNs, so there is no printed value to compare with).
# What pins it is the mathematics of the subproblems it solves (stationarity, monotone descent, the g = 1 special case).
#   module: y = W2 (SiLU(Wg x) * (Wu x)).  Only the "up" branch is split: Z = z_u with Z ~ Wu X, A ~ g * Z, where
#   g = SiLU(Wg_0 X) is computed once from the pre-trained gate and kept fixed; the gate weights are only row-masked.
#   With g fixed, phi(z) = g z is linear, so every subproblem of the FFN objective of Appendix A.1 keeps its closed
#   form: the weight recoveries and the a-update are unchanged (phi(Z) = g Z), the z-update is one quadratic.
# --------------------------------------------------------------------------------------------------
def silu(x):
    x = np.asarray(x, F64)
    return x / (1.0 + np.exp(-x))


def swiglu_init(X, Wg_0, Wu_0, W2_0, dual_mode=False):
    """Initialisation of a SwiGLU module: g = SiLU(Wg_0 X) (fixed), Z = Wu_0 X, A = g Z, Ypre = W2_0 A, and the
    accumulators of the first weight recovery.  Returns (state with .gate = g, Ypre)."""
    X = np.asarray(X, F64)
    g = silu(np.asarray(Wg_0, F64) @ X)
    Zpre = np.asarray(Wu_0, F64) @ X
    Apre = g * Zpre
    Ypre = np.asarray(W2_0, F64) @ Apre
    st = FfnState(
        Z=Zpre.copy(), U=np.zeros_like(Zpre) if dual_mode else None,
        G_X=X @ X.T, G_A=Apre @ Apre.T, R1=Zpre @ X.T, R2=Ypre @ Apre.T, absA=np.abs(Apre).sum(axis=1), gate=g)
    return st, Ypre


def swiglu_zu_update(A, g, z1u, alpha, beta, U=None):
    """argmin_zu beta (a + u - g zu)^2 + alpha (zu - z1u)^2 for a gated unit a = g * zu, g = SiLU(gate)."""
    Au = np.asarray(A, F64) + (0.0 if U is None else np.asarray(U, F64))
    return (beta * g * Au + alpha * z1u) / (beta * g * g + alpha)


# --------------------------------------------------------------------------------------------------
# Multi-head attention, Method 2 (Appendix A, "Computation on Multi-Head Attention layers"; Algorithm 2, SparseLLM2)
#
# One attention module on one sequence of T tokens (columns of X in R^{d x T}); h heads of width d_h = d / h; head i
# owns rows [i d_h, (i+1) d_h) of W_Q X, W_K X, W_V X.  Forward definition (paper, per head):
#     S_i = Q_i^T K_i / sqrt(d_h)  (T x T, rows = queries),  P_i = softmax over the keys of each row of S_i,
#     head_i = V_i P_i^T  (d_h x T),  a^attn = Concat_i head_i  (d x T),  z_{l+1}^pre = W_O a^attn.
# Readings (the section is printed with inconsistent shapes; none of these choices is fixed by the paper):
#   * Method 2's last two terms are printed as |z_l - (M^Q.W^Q) a_{l-1}|^2 + |z_l - (M^K.W^K) a_{l-1}|^2 with one z_l,
#     which cannot equal two different d x T products, while z_l is also the T x T argument of the softmax.  Read as
#     "separate constraints for the Q and K projections": the auxiliary output z_l is the PAIR (Zq, Zk) with
#     Zq ~ W_Q X, Zk ~ W_K X, and the softmax term sees the logits S(Zq, Zk).  Each projection then has the linear
#     recovery W = z a^+ that Algorithm 2 runs "for W_Q, W_K, W_V, W_O separately".
#   * a_l is the attention-probability tensor P (one T x T matrix per head), a^attn_l the concatenated head outputs.
#   * Eq. (85) [a_l] is quadratic in P; the paper prescribes gradient steps: `a_steps` steps of plain gradient descent
#     with the step 1 / L, L = 2 (alpha |V_i|_F^2 + beta) >= the largest curvature of that quadratic (so every step
#     descends), per head.
#   * Eq. (86) [a^attn_l] is an unconstrained quadratic with the closed-form minimiser
#     (W_O^T W_O + I)^-1 (W_O^T z_{l+1}^pre + Concat_i V_i P_i^T); the paper names no solver for it, the minimiser is used.
#   * Eq. (87) [z_l] goes through the softmax: `z_steps` steps of gradient descent on (Zq, Zk) jointly with the step
#     eta_z / (2 alpha + beta (|Zq_i|_F^2 + |Zk_i|_F^2) / d_h) per head (a bound on the Gauss-Newton curvature of the
#     softmax term plus the curvature 2 alpha of the quadratic terms), eta_z <= 1.
#   * The elementwise "if z < 0" select that Algorithm 2 repeats inside SparseLLM2 belongs to the ReLU module and has
#     no counterpart for a softmax; it is not applied.
#   * causal = True masks keys after the query (the decoder models the paper prunes are causal; the printed formulas
#     omit the mask "for clarity").
# The paper prints no numbers for this path; what pins the code below is mathematics (tests/test_oracle_mha_pins.py):
# the forward definition as plain loops, central differences of both gradients, stationarity of the closed form,
# convergence of the Eq. (85) steps to the linear-solve minimiser, descent of every sub-step, and special cases.
# --------------------------------------------------------------------------------------------------
@dataclasses.dataclass
class MhaParams:
    n_heads: int = 1
    alpha: float = 1.0
    beta: float = 1.0
    a_steps: int = 4
    z_steps: int = 4
    eta_z: float = 1.0
    causal: bool = True


def softmax_rows(S, causal=False):
    """Row-wise softmax of a T x T logit matrix; with `causal`, key u > query t gets probability 0."""
    S = np.asarray(S, F64)
    if causal:
        T = S.shape[-1]
        S = np.where(np.tril(np.ones((T, T), bool)), S, -np.inf)
    E = np.exp(S - S.max(axis=-1, keepdims=True))
    return E / E.sum(axis=-1, keepdims=True)


def mha_logits(Zq_i, Zk_i):
    """S_i = Q_i^T K_i / sqrt(d_h) for one head (inputs d_h x T, tokens are columns)."""
    return np.asarray(Zq_i, F64).T @ np.asarray(Zk_i, F64) / math.sqrt(np.shape(Zq_i)[0])


def mha_forward(X, Wq, Wk, Wv, Wo, n_heads, causal=True):
    """The attention module as the paper defines it, on one sequence.  Returns (Zq, Zk, V, P [h, T, T], Aattn, Y)."""
    X = np.asarray(X, F64)
    d, T = X.shape
    dh = d // n_heads
    Zq, Zk, V = np.asarray(Wq, F64) @ X, np.asarray(Wk, F64) @ X, np.asarray(Wv, F64) @ X
    P = np.zeros((n_heads, T, T), F64)
    A = np.zeros((d, T), F64)
    for i in range(n_heads):
        r = slice(i * dh, (i + 1) * dh)
        P[i] = softmax_rows(mha_logits(Zq[r], Zk[r]), causal)
        A[r] = V[r] @ P[i].T
    return Zq, Zk, V, P, A, np.asarray(Wo, F64) @ A


def mha_heads(V, P, n_heads):
    """Concat_i V_i P_i^T (d x T)."""
    d = V.shape[0]
    dh = d // n_heads
    return np.concatenate([V[i * dh:(i + 1) * dh] @ P[i].T for i in range(n_heads)], axis=0)


def mha_objective(X, Ypre, Wq, Wk, Wv, Wo, Zq, Zk, P, Aattn, p):
    """Method 2 objective on one sequence; returns its five terms in the printed order."""
    X = np.asarray(X, F64)
    V = np.asarray(Wv, F64) @ X
    dh = X.shape[0] // p.n_heads
    t1 = p.alpha * ((np.asarray(Ypre, F64) - np.asarray(Wo, F64) @ Aattn) ** 2).sum()
    t2 = p.alpha * ((Aattn - mha_heads(V, P, p.n_heads)) ** 2).sum()
    t3 = 0.0
    for i in range(p.n_heads):
        r = slice(i * dh, (i + 1) * dh)
        t3 += p.beta * ((P[i] - softmax_rows(mha_logits(Zq[r], Zk[r]), p.causal)) ** 2).sum()
    t4 = p.alpha * ((Zq - np.asarray(Wq, F64) @ X) ** 2).sum()
    t5 = p.alpha * ((Zk - np.asarray(Wk, F64) @ X) ** 2).sum()
    return np.array([t1, t2, t3, t4, t5], F64)


def mha_a_objective_grad(P_i, A_i, V_i, Phi_i, alpha, beta):
    """Eq. (85) for one head: f(P) = alpha |A_i - V_i P^T|^2 + beta |P - Phi_i|^2 and its gradient in P."""
    R = A_i - V_i @ P_i.T
    f = alpha * (R ** 2).sum() + beta * ((P_i - Phi_i) ** 2).sum()
    g = -2.0 * alpha * (R.T @ V_i) + 2.0 * beta * (P_i - Phi_i)
    return f, g


def mha_a_update(P, Aattn, V, Zq, Zk, p):
    """`a_steps` gradient steps of Eq. (85) on every head's P_i with the step 1 / (2 (alpha |V_i|_F^2 + beta))."""
    dh = V.shape[0] // p.n_heads
    P = P.copy()
    for i in range(p.n_heads):
        r = slice(i * dh, (i + 1) * dh)
        Phi = softmax_rows(mha_logits(Zq[r], Zk[r]), p.causal)
        step = 1.0 / (2.0 * (p.alpha * (V[r] ** 2).sum() + p.beta))
        for _ in range(p.a_steps):
            _, g = mha_a_objective_grad(P[i], Aattn[r], V[r], Phi, p.alpha, p.beta)
            P[i] = P[i] - step * g
    return P


def mha_attn_update(Ypre, Wo, Hd):
    """Minimiser of Eq. (86): a^attn = (W_O^T W_O + I)^-1 (W_O^T z_{l+1}^pre + Hd), Hd = Concat_i V_i P_i^T
    (alpha multiplies both terms and drops out)."""
    Wo = np.asarray(Wo, F64)
    d = Wo.shape[1]
    return np.linalg.solve(Wo.T @ Wo + np.eye(d), Wo.T @ np.asarray(Ypre, F64) + Hd)


def mha_z_objective_grad(Zq_i, Zk_i, P_i, Tq_i, Tk_i, alpha, beta, causal):
    """Eq. (87) for one head: f = beta |P_i - softmax(S(Zq, Zk))|^2 + alpha |Zq - Tq|^2 + alpha |Zk - Tk|^2 with the
    targets Tq = (W_Q X)_i, Tk = (W_K X)_i; returns (f, df/dZq, df/dZk).  Softmax backward written out:
    dS = 2 beta Phi * (E - rowsum(E * Phi)), E = Phi - P."""
    dh = Zq_i.shape[0]
    Phi = softmax_rows(mha_logits(Zq_i, Zk_i), causal)
    E = Phi - P_i
    f = beta * (E ** 2).sum() + alpha * ((Zq_i - Tq_i) ** 2).sum() + alpha * ((Zk_i - Tk_i) ** 2).sum()
    dS = 2.0 * beta * Phi * (E - (E * Phi).sum(axis=1, keepdims=True))
    gq = Zk_i @ dS.T / math.sqrt(dh) + 2.0 * alpha * (Zq_i - Tq_i)
    gk = Zq_i @ dS / math.sqrt(dh) + 2.0 * alpha * (Zk_i - Tk_i)
    return f, gq, gk


def mha_z_step_size(Zq_i, Zk_i, alpha, beta, eta_z):
    dh = Zq_i.shape[0]
    return eta_z / (2.0 * alpha + beta * ((Zq_i ** 2).sum() + (Zk_i ** 2).sum()) / dh)


def mha_z_update(Zq, Zk, P, Tq, Tk, p):
    """`z_steps` joint gradient steps of Eq. (87) on (Zq_i, Zk_i) of every head; the step is recomputed from the
    current iterate before each step."""
    dh = Zq.shape[0] // p.n_heads
    Zq, Zk = Zq.copy(), Zk.copy()
    for i in range(p.n_heads):
        r = slice(i * dh, (i + 1) * dh)
        for _ in range(p.z_steps):
            _, gq, gk = mha_z_objective_grad(Zq[r], Zk[r], P[i], Tq[r], Tk[r], p.alpha, p.beta, p.causal)
            step = mha_z_step_size(Zq[r], Zk[r], p.alpha, p.beta, p.eta_z)
            Zq[r], Zk[r] = Zq[r] - step * gq, Zk[r] - step * gk
    return Zq, Zk


def mha_step(X, Ypre, Wq, Wk, Wv, Wo, Zq, Zk, P, Aattn, p):
    """The auxiliary-variable updates of one outer step of SparseLLM2 on one sequence, weights fixed, in the order of
    Algorithm 2: Eq. (85) a_l = P, Eq. (86) a^attn_l, Eq. (87) z_l = (Zq, Zk).  Returns (Zq, Zk, P, Aattn)."""
    X = np.asarray(X, F64)
    V = np.asarray(Wv, F64) @ X
    P = mha_a_update(P, Aattn, V, Zq, Zk, p)
    Aattn = mha_attn_update(Ypre, Wo, mha_heads(V, P, p.n_heads))
    Zq, Zk = mha_z_update(Zq, Zk, P, np.asarray(Wq, F64) @ X, np.asarray(Wk, F64) @ X, p)
    return Zq, Zk, P, Aattn


def mha_recover_weights(Xs, Ys, Zqs, Zks, As, head_mask, d_head, rho, rho_relative=True):
    """Weight recovery of one outer step of SparseLLM2 ("prune by importance + recovery solver, do for W_Q, W_K, W_V,
    W_O separately") from the auxiliary variables of all sequences (lists, tokens as columns), for the projections
    whose recovery is linear in them:
      W_Q = Zq X^+ and W_K = Zk X^+ as ridge solves on G_X = sum X X^T, rows of pruned heads set to zero (for a row
      mask the restricted solution is the row-masked one);  W_O = Ypre Aattn^+ on the columns of the kept heads
      (restricted ridge solve, ridge of the full system), other columns zero.
    Returns (W_Q, W_K, W_O)."""
    d = Xs[0].shape[0]
    G_X = sum(X @ X.T for X in Xs)
    R_Q = sum(Zq @ X.T for Zq, X in zip(Zqs, Xs))
    R_K = sum(Zk @ X.T for Zk, X in zip(Zks, Xs))
    G_A = sum(A @ A.T for A in As)
    R_O = sum(Y @ A.T for Y, A in zip(Ys, As))
    keep = np.repeat(np.asarray(head_mask).astype(bool), d_head)
    rho1 = effective_ridge(G_X, rho, rho_relative)
    Wq = np.where(keep[:, None], ridge_solve(R_Q, G_X, rho1), 0.0)
    Wk = np.where(keep[:, None], ridge_solve(R_K, G_X, rho1), 0.0)
    Wo = restricted_refit(R_O, G_A, keep, effective_ridge(G_A, rho, rho_relative))
    return Wq, Wk, Wo


def mha_recover_value_weights(Xs, Ps, As, head_mask, d_head, rho, rho_relative=True):
    """Recovery of W_V ("W = z a^+", done "for W_Q, W_K, W_V, W_O separately") from the auxiliary variables of all
    sequences.  The second term of the Method 2 objective ties head i's rows of a^attn to W_V through
        a^attn_i = W_V,i X P_i^T        (d_h x T per sequence, tokens as columns),
    so the regressors of head i are R_i = X P_i^T (d x T) and its least-squares recovery over all sequences s is
        W_V,i = (sum_s A_i,s R_i,s^T) (sum_s R_i,s R_i,s^T + rho_i I)^-1,
    one ridge system per head (rho_i relative to the mean diagonal of that head's Gram matrix when rho_relative).
    Rows of pruned heads are zero.  Xs: list of [d, T]; Ps: list of [h, T, T]; As: list of [d, T]."""
    d = Xs[0].shape[0]
    h = len(head_mask)
    Wv = np.zeros((d, d), F64)
    for i in range(h):
        if not head_mask[i]:
            continue
        r = slice(i * d_head, (i + 1) * d_head)
        G = np.zeros((d, d), F64)
        C = np.zeros((d_head, d), F64)
        for X, P, A in zip(Xs, Ps, As):
            R = np.asarray(X, F64) @ np.asarray(P[i], F64).T
            G += R @ R.T
            C += np.asarray(A, F64)[r] @ R.T
        Wv[r] = ridge_solve(C, G, effective_ridge(G, rho, rho_relative))
    return Wv
