"""sp_struct_scores_static: the Wanda score call for callers that cannot allocate device memory.

Some users of the library run where no allocation is possible at call time (device memory handed out once at
start-up, or a pipeline that must not be stalled by an allocation's device-wide synchronisation).  For them the library
carries a fixed 2 MiB scratch array of its own, and this entry point takes inputs and outputs only.  The test calls it
through the C ABI twice in a row, with different sizes, so that the second call runs on scratch the first one left
dirty, and checks both results against sp_struct_scores (caller workspace) on the same inputs.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import struprune_oracle as O
from paper_2510_03246_b200 import api, synth
from tests._util import np64, relerr

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(d, n_units, group, N, seed):
    n = n_units * group
    W = (synth.standard_variates(seed, 1, d * n, "gauss").view(d, n)).to(DEV)
    A = synth.standard_variates(seed, 2, N * n, "gauss").view(N, n).double()
    colsq = (A ** 2).sum(0).float().to(DEV)
    colabs = A.abs().sum(0).to(DEV)
    return W, colsq, colabs


def _static_call(kind, n_units, group, W, colsq, colabs, N):
    scores = torch.full((n_units,), float("nan"), dtype=torch.float32, device=DEV)
    imp = torch.full((1,), float("nan"), dtype=torch.float64, device=DEV)
    api.sp_struct_scores_static(kind, n_units, scores, imp, group=group, W=W, colsq=colsq, colabs=colabs,
                                inv_tokens=1.0 / N)
    return scores, imp


def test_static_scores_match_workspace_scores_on_two_calls_in_a_row():
    # first call: wide (few row blocks of partial sums); second call: narrow and ragged (many row blocks), so it reuses
    # the part of the scratch array the first call filled with other values
    cases = [(api.SP_SCORE_WANDA_L2, 300, 2500, 1, 40, 11), (api.SP_SCORE_WANDA_L1, 777, 37, 4, 64, 12)]
    for kind, d, n_units, group, N, seed in cases:
        W, colsq, colabs = _inputs(d, n_units, group, N, seed)
        got_s, got_i = _static_call(kind, n_units, group, W, colsq, colabs, N)
        ref_s, ref_i, _ = api.sp_struct_scores(kind, n_units, group, W=W, colsq=colsq, colabs=colabs,
                                               inv_tokens=1.0 / N)
        torch.cuda.synchronize()
        # same kernels and the same fixed reduction order: the tolerance of the score parity tests is met with room
        assert relerr(np64(got_s), np64(ref_s)) < 1e-6
        assert abs(got_i.item() - ref_i.item()) <= 1e-6 * abs(ref_i.item())
        assert np.array_equal(got_s.cpu().numpy(), ref_s.cpu().numpy())


def test_static_scores_units_that_straddle_column_groups_and_unaligned_weights():
    """Units whose width does not divide the kernel's 128-column groups (3 and 96 columns per unit) take the path that
    gathers a unit's column values across groups; a weight view with a pitch larger than its width and a start that is
    not 16-byte aligned takes the scalar loads.  Each runs right after a call that left other values in the scratch,
    and is also checked against the oracle's scores of the same inputs."""
    first = _inputs(300, 2500, 1, 40, 21)
    _static_call(api.SP_SCORE_WANDA_L2, 2500, 1, *first, 40)            # dirties the scratch
    for kind, d, n_units, group, N, seed in ((api.SP_SCORE_WANDA_L2, 210, 333, 3, 50, 22),
                                             (api.SP_SCORE_WANDA_L1, 130, 21, 96, 32, 23)):
        n = n_units * group
        W, colsq, colabs = _inputs(d, n_units, group, N, seed)
        wide = torch.zeros(d, n + 5, device=DEV)
        wide[:, 1:n + 1] = W
        Wv = wide[:, 1:n + 1]                                            # pitch n + 5, first element 4 bytes in
        for Wm in (W, Wv):
            got_s, got_i = _static_call(kind, n_units, group, Wm, colsq, colabs, N)
            ref_s, ref_i, _ = api.sp_struct_scores(kind, n_units, group, W=Wm, colsq=colsq, colabs=colabs,
                                                   inv_tokens=1.0 / N)
            torch.cuda.synchronize()
            assert np.array_equal(got_s.cpu().numpy(), ref_s.cpu().numpy())
            assert abs(got_i.item() - ref_i.item()) <= 1e-12 * abs(ref_i.item())
            if kind == api.SP_SCORE_WANDA_L2:
                want, want_i = O.wanda_scores(np64(W), colsq=np64(colsq), kind="l2", group=group)
            else:
                want, want_i = O.wanda_scores(np64(W), colabs_mean=np64(colabs) / N, kind="l1", group=group)
            assert relerr(np64(got_s), want) < 1e-6 and abs(got_i.item() - want_i) < 1e-6 * abs(want_i)


def test_static_scores_reject_sizes_beyond_the_builtin_scratch():
    n_units = api.STATIC_SCORES_MAX_COLS + 8
    W = torch.zeros(2, n_units, device=DEV)
    colsq = torch.zeros(n_units, device=DEV)
    scores = torch.zeros(n_units, device=DEV)
    imp = torch.zeros(1, dtype=torch.float64, device=DEV)
    with pytest.raises(api.SpError) as e:
        api.sp_struct_scores_static(api.SP_SCORE_WANDA_L2, n_units, scores, imp, W=W, colsq=colsq)
    assert e.value.code == 10 and "static scratch" in str(e.value)
    with pytest.raises(api.SpError) as e:       # Lemma-1 streaming has no static-scratch variant
        api.sp_struct_scores_static(api.SP_SCORE_LEMMA1, 8, scores, imp, W=W[:, :8], colsq=colsq)
    assert e.value.code == 9
