"""World-size-2 gloo test of the multi-GPU plumbing (runs on CPU)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_03246_b200 import parallel


def _worker(rank, world, port, L):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = parallel.layers_of_rank(L, rank, world)
        local = {l: 1.0 + 0.25 * l for l in mine}
        full = parallel.gather_importances(local, L)
        assert torch.allclose(full, 1.0 + 0.25 * torch.arange(L, dtype=torch.float64))
        assert parallel.max_over_ranks(float(rank + 1)) == float(world)
        assert parallel.sum_over_ranks(float(len(mine))) == float(L)
    finally:
        dist.destroy_process_group()


def test_layer_sharding_is_a_partition():
    for L in (1, 7, 24, 32):
        for world in (1, 2, 3, 8):
            owned = [parallel.layers_of_rank(L, r, world) for r in range(world)]
            flat = sorted(x for o in owned for x in o)
            assert flat == list(range(L))
            assert max(len(o) for o in owned) - min(len(o) for o in owned) <= 1


def test_importance_gather_world2():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, 7), nprocs=2, join=True)


# ------------------------------------------------------------------------------------------------ token sharding
# The token-sharded loop is host logic around the module calls; here an oracle-backed stand-in plays the module, so
# that what is summed, when, and what is broadcast can be checked on CPU against the oracle run over all tokens.
import copy

import numpy as np

from oracle import struprune_oracle as O
from paper_2510_03246_b200 import api, synth

_TS_CFG = synth.scaled(synth.CONFIGS["C1"], d=24, n=56, tokens=600)
_TS_K, _TS_ITERS = 20, 3


class _OracleShard:
    """One token shard of an FFN module with the interface the sharded loop uses (tensors it sums are torch CPU)."""

    def __init__(self, X, W1_0, W2_0, kind):
        self.X, self.W1_0, self.W2_0, self.kind = X, W1_0, W2_0, kind
        d, n = X.shape[0], W1_0.shape[0]
        z = lambda *s: torch.zeros(*s, dtype=torch.float64)
        self.G_X, self.G_A, self.R1, self.R2, self.absA = z(d, d), z(n, n), z(n, d), z(d, n), z(n)
        self.scores, self.mask = z(n), torch.ones(n, dtype=torch.uint8)
        self.report = z(len(api.REPORT_FIELDS))
        self.report_fields = api.REPORT_FIELDS

    def _put(self, st):
        for name in ("G_X", "G_A", "R1", "R2", "absA"):
            getattr(self, name).copy_(torch.from_numpy(np.ascontiguousarray(getattr(st, name))))

    def _state(self):
        return O.FfnState(Z=self.Z, U=None, G_X=self.G_X.numpy().copy(), G_A=self.G_A.numpy().copy(),
                          R1=self.R1.numpy().copy(), R2=self.R2.numpy().copy(), absA=self.absA.numpy().copy(),
                          mask=self.mask.numpy().copy())

    def _params(self, p):
        return O.AdmmParams(rho=p.rho, k_keep=p.k_keep, score_kind=self.kind, reselect_mask=bool(p.reselect_mask),
                            refit=bool(p.refit))

    def sp_ffn_init(self):
        st, self.Ypre = O.ffn_init(self.X, self.W1_0, self.W2_0)
        self.Z = st.Z
        self._put(st)

    def sp_admm_scores(self, p):
        s, _ = O.admm_weight_phase(self._state(), self.W1_0, self._params(p), self.X.shape[1])
        self.scores.copy_(torch.from_numpy(s))

    def select_mask(self, k):
        self.mask.copy_(torch.from_numpy(O.topk_mask(self.scores.numpy(), k)[0]))

    def sp_admm_step(self, p):
        assert not p.reselect_mask
        st = self._state()
        _, _, rep, _ = O.admm_step(st, self.X, self.Ypre, self.W1_0, self._params(p))
        self.Z, self.W1, self.W2 = st.Z, st.W1, st.W2
        self._put(st)
        self.report.copy_(torch.tensor([float(rep.get(k, float("nan"))) for k in api.REPORT_FIELDS],
                                       dtype=torch.float64))


def _ts_inputs():
    X = synth.make_activations(_TS_CFG, 0).double().numpy().T          # d x N
    W1, W2 = (w.double().numpy() for w in synth.make_weights(_TS_CFG, 0))
    return X, W1, W2


def _ts_reference(kind):
    X, W1, W2 = _ts_inputs()
    st, Y = O.ffn_init(X, W1, W2)
    p = O.AdmmParams(rho=_TS_CFG.rho, k_keep=_TS_K, score_kind=kind)
    reps = []
    for _ in range(_TS_ITERS):
        reps.append(O.admm_step(st, X, Y, W1, p)[2])
    return st, reps


def _ts_check(lead, reports, kind):
    st, reps = _ts_reference(kind)
    assert np.array_equal(lead.mask.numpy(), st.mask)
    for name in ("W1", "W2"):
        ref = getattr(st, name)
        assert np.abs(getattr(lead, name) - ref).max() <= 1e-9 * np.abs(ref).max(), name
    for name in ("G_A", "R1", "R2", "absA"):
        ref = getattr(st, name)
        assert np.abs(getattr(lead, name).numpy() - ref).max() <= 1e-9 * np.abs(ref).max(), name
    for got, ref in zip(reports, reps):
        for key in ("res_act", "res_in", "res_out"):
            assert abs(got[key] - ref[key]) <= 1e-9 * max(abs(ref[key]), 1e-30), key


def _ts_worker(rank, world, port, kind):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        X, W1, W2 = _ts_inputs()
        cut = [0, 350, X.shape[1]]                                       # unequal shards
        shard = _OracleShard(X[:, cut[rank]:cut[rank + 1]], W1, W2, kind)
        parallel.token_sharded_init([shard])
        p = api.AdmmParams(rho=_TS_CFG.rho, k_keep=_TS_K)
        reports = parallel.token_sharded_iterations([shard], p, _TS_ITERS)
        _ts_check(shard, reports, kind)                                  # every rank holds the full result
    finally:
        dist.destroy_process_group()


def test_token_sharded_iterations_world2_equal_the_unsharded_run():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_ts_worker, args=(2, port, "wanda_l2"), nprocs=2, join=True)


def test_token_sharded_iterations_three_local_shards():
    """The same loop with three shards held by one process (no process group): sums over the local list."""
    for kind in ("wanda_l2", "lemma1"):
        X, W1, W2 = _ts_inputs()
        cut = [0, 100, 390, X.shape[1]]
        shards = [_OracleShard(X[:, cut[i]:cut[i + 1]], W1, W2, kind) for i in range(3)]
        parallel.token_sharded_init(shards)
        reports = parallel.token_sharded_iterations(shards, api.AdmmParams(rho=_TS_CFG.rho, k_keep=_TS_K), _TS_ITERS)
        for sh in shards:
            assert torch.equal(sh.mask, shards[0].mask) and torch.equal(sh.G_A, shards[0].G_A)
        _ts_check(shards[0], reports, kind)
