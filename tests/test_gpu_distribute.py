"""Steps 1 and 2 of the "-distribute" variant of Algorithm 1 on the GPU against the oracle: slice statistics of the
weights (per attention head over W_Q, W_K, W_V rows and W_O columns; per MLP matrix), the importances with depth decay
and attention/MLP ratio, and the inverse-weighted allocation of both module groups."""
import numpy as np
import pytest
import torch

from oracle import struprune_oracle as O
from paper_2510_03246_b200 import api, pipeline, synth
from tests._util import np64

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _w(shape, seed, tid, scale=0.02):
    n = int(np.prod(shape))
    return (synth.standard_variates(seed, tid, n, "gauss").view(*shape) * scale + 0.003)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,cols,axis,group", [(96, 80, 0, 24), (96, 80, 1, 20), (96, 80, 1, 10), (50, 33, 0, 0),
                                                  (2048, 1024, 1, 64), (300, 7, 0, 100)])
def test_weight_stats_slices(dtype, rows, cols, axis, group):
    big = _w((rows, cols + 5), 3, rows + cols).to(dtype)
    W = big[:, :cols]                      # a leading dimension larger than the width
    Wg = big.to(DEV)[:, :cols]
    st = api.sp_weight_stats(Wg, axis, group).cpu().numpy()
    Wd = np64(W.float())
    nb = 1 if group == 0 else (rows // group if axis == 0 else cols // group)
    assert st.shape == (nb, 4)
    for b in range(nb):
        blk = Wd if group == 0 else (Wd[b * group:(b + 1) * group] if axis == 0 else Wd[:, b * group:(b + 1) * group])
        want = np.array([np.abs(blk).sum(), blk.sum(), (blk * blk).sum(), blk.size])
        # the kernel adds up to 64 values in fp32 before it goes to fp64: each such partial sum carries at most 64
        # roundings of 2^-24 relative to the sum of magnitudes
        tol = np.array([1, 1, np.abs(blk).max(), 0]) * (64 * 2.0 ** -24) * np.abs(blk).sum() + 1e-300
        assert np.all(np.abs(st[b] - want) <= tol), (b, st[b], want)
    # accumulation adds to what is there
    st2 = api.sp_weight_stats(Wg, axis, group, api.sp_weight_stats(Wg, axis, group), accumulate=True).cpu().numpy()
    assert np.allclose(st2, 2 * st, rtol=1e-14)


def test_weight_stats_argument_errors():
    W = torch.zeros(12, 8, device=DEV)
    with pytest.raises(api.SpError) as e:
        api.sp_weight_stats(W, 0, 5)
    assert e.value.code == 2


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_plan_distribute_matches_oracle(dtype):
    L, H, d, n = 5, 6, 96, 160
    dh = d // H

    def host_layer(l):
        s = 0.02 * (1.0 + 0.3 * l)
        return dict(Wq=_w((d, d), 40 + l, 1, s), Wk=_w((d, d), 40 + l, 2, s), Wv=_w((d, d), 40 + l, 3, s),
                    Wo=_w((d, d), 40 + l, 4, s), fc1=_w((n, d), 40 + l, 5, s), fc2=_w((d, n), 40 + l, 6, s))

    host = [{k: v.to(dtype) for k, v in host_layer(l).items()} for l in range(L)]
    rho, gamma, rbar, T_rel = 1.7, 0.93, 0.5, 0.05
    plan = pipeline.plan_distribute(lambda l: {k: v.to(DEV) for k, v in host[l].items()}, L, H, n, rbar, T_rel=T_rel,
                                    rho=rho, gamma=gamma, device=DEV)
    layers64 = [{k: np64(v.float()) for k, v in w.items()} for w in host]
    Ia, Im = O.distribute_importance(layers64, H, dh, rho, gamma)
    assert np.allclose(np64(plan["I_attn"]), Ia, rtol=2e-6) and np.allclose(np64(plan["I_mlp"]), Im, rtol=2e-6)
    for key, I, units, kname in (("attn", Ia, H, "k_heads"), ("mlp", Im, n, "k_channels")):
        r, k = O.allocate_sparsity(I, np.full(L, units), rbar, T_rel * np.abs(I).mean(), "inverse")
        # the allocation is compared on the GPU's own importances (fp64 on both sides)
        r, k = O.allocate_sparsity(np64(plan["I_" + key]), np.full(L, units), rbar,
                                   T_rel * np.abs(np64(plan["I_" + key])).mean(), "inverse")
        assert np.abs(np64(plan["r_" + key]) - r).max() < 1e-9
        frac = r * units + 0.5
        safe = np.abs(frac - np.round(frac)) > 1e-6
        assert np.array_equal(plan[kname].cpu().numpy()[safe], k[safe])
    # the two groups are normalised separately: each keeps its own mean pruned fraction
    assert abs(np64(plan["r_attn"]).mean() - rbar) < 1e-9 and abs(np64(plan["r_mlp"]).mean() - rbar) < 1e-9
