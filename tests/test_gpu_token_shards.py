"""Token sharding inside one module on the GPU: two shards held by one process (their kernels run one after the other
on one stream; the sums that NCCL would do across GPUs are done over the local list), against the oracle run over all
tokens and against the unsharded module."""
import numpy as np
import pytest
import torch

from oracle import struprune_oracle as O
from paper_2510_03246_b200 import api, parallel, synth
from tests._util import TOL, np64, relerr

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("storage,kind", [("f32", "wanda_l2"), ("f32", "lemma1"), ("bf16", "wanda_l2")])
def test_two_token_shards_equal_the_unsharded_module(storage, kind):
    base = synth.CONFIGS["C1" if storage == "f32" else "C2"]
    cfg = synth.scaled(base, d=96, n=328, tokens=1000, sparsity=0.5, outlier_frac=0.02)
    kinds = {"wanda_l2": api.SP_SCORE_WANDA_L2, "lemma1": api.SP_SCORE_LEMMA1}
    X = synth.make_activations(cfg, 0)
    W1, W2 = synth.make_weights(cfg, 0)
    k, iters, cut = cfg.k_keep, 3, 616                               # unequal shards, the second not a multiple of 8
    shards = [api.FfnModule(X[a:b].to(DEV), W1.to(DEV), W2.to(DEV), token_chunk=256) for a, b in ((0, cut), (cut, 1000))]
    parallel.token_sharded_init(shards)
    p = api.AdmmParams(rho=cfg.rho, k_keep=k, score_kind=kinds[kind], token_chunk=256)
    reports = parallel.token_sharded_iterations(shards, p, iters)
    torch.cuda.synchronize()
    for m in shards:
        m.check_status()
    assert torch.equal(shards[0].mask, shards[1].mask) and torch.equal(shards[0].G_A, shards[1].G_A)
    tol = TOL[X.dtype]
    # the unsharded module through the ordinary step
    full = api.FfnModule(X.to(DEV), W1.to(DEV), W2.to(DEV), token_chunk=256)
    full.sp_ffn_init()
    for _ in range(iters):
        full.sp_admm_step(p)
    torch.cuda.synchronize()
    full.check_status()
    same_mask = torch.equal(full.mask, shards[0].mask)
    if storage == "f32":
        # the oracle over all tokens, free-running over the same iterations (in bf16 storage free-running runs drift
        # apart by the storage rounding of every iteration; there the unsharded module below is the comparison)
        Xo = np64(X).T
        st, Y = O.ffn_init(Xo, np64(W1), np64(W2))
        p_or = O.AdmmParams(rho=cfg.rho, k_keep=k, score_kind=kind)
        for _ in range(iters):
            rep_or = O.admm_step(st, Xo, Y, np64(W1), p_or)[2]
        assert same_mask and np.array_equal(shards[0].mask.cpu().numpy(), st.mask)
        loose = tol * 10                                              # three free-running iterations
        assert relerr(np64(shards[0].W1), st.W1) < loose and relerr(np64(shards[0].W2), st.W2) < loose
        assert relerr(np64(shards[0].G_A), st.G_A) < loose and relerr(np64(shards[0].R2), st.R2) < loose
        Z = np.concatenate([np64(m.Z).T for m in shards], axis=1)
        assert relerr(Z, st.Z) < loose
        assert abs(reports[-1]["res_act"] - rep_or["res_act"]) <= 10 * loose * reports[-1]["a_sq"]
    elif not same_mask:
        # the two runs round differently: they may only disagree on units whose scores sit at the threshold
        sc = np64(full.scores)
        tau = np.sort(sc)[::-1][k - 1]
        diff = np.flatnonzero(full.mask.cpu().numpy() != shards[0].mask.cpu().numpy())
        assert np.all(np.abs(sc[diff] - tau) <= 10 * tol * np.abs(sc).max())
    if same_mask:
        assert relerr(np64(shards[0].W1), np64(full.W1)) < 10 * tol
        assert relerr(np64(shards[0].W2), np64(full.W2)) < 10 * tol
        assert relerr(np64(shards[0].G_A), np64(full.G_A)) < 10 * tol
    assert int(shards[0].mask.sum()) == k
