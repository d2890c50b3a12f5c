"""CPU-only checks of the boundary: libsp.so builds, loads, exports every symbol include/sp.h declares, and its
host-side argument validation returns the documented codes before anything is launched."""
import ctypes as C
import os
import re

import pytest

from paper_2510_03246_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sp_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_symbols()
    assert {"sp_gram_accumulate", "sp_admm_step", "sp_struct_scores", "sp_allocate_sparsity",
            "sp_apply_mask"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in sp.h but not exported by libsp.so"
    assert set(api.EXPORTS) == set(names)


def test_version_and_status_strings(lib):
    assert lib.sp_version() >= 100
    assert api.status_string(0) == "ok"
    assert "workspace" in api.status_string(5)
    assert "positive definite" in api.status_string(6)


def test_workspace_queries(lib):
    small = api.workspace_bytes(api.SP_WS_ADMM_STEP, 96, 328, 600, 0, api.SP_F32)
    big = api.workspace_bytes(api.SP_WS_ADMM_STEP, 2048, 8192, 262144, 16384, api.SP_BF16)
    assert 0 < small < big < 8 << 30
    # the fp64 solve holds the system in doubles; the fp32 solve adds the bf16 parts of the factor instead
    w64 = api.workspace_bytes(api.SP_WS_RIDGE_SOLVE, 64, 128, 0, 0, api.SP_F64)
    w32 = api.workspace_bytes(api.SP_WS_RIDGE_SOLVE, 64, 128, 0, 0, api.SP_F32)
    assert w64 >= 8 * 128 * 128 and w32 >= 4 * 128 * 128 + 6 * 128 * 128
    assert api.workspace_bytes(99, 1, 1, 1) == 0


def test_host_side_validation_without_gpu(lib):
    fake = C.c_void_p(0x1000)   # never dereferenced: every call below must fail before any launch
    # sp_apply_mask: k_keep > n_units
    assert lib.sp_apply_mask(fake, 10, 11, 1, fake, None, None, None, None, None, 0, None) == 2
    assert lib.sp_apply_mask(None, 10, 5, 1, fake, None, None, None, None, None, 0, None) == 1
    # sp_allocate_sparsity: bad temperature / layer count
    assert lib.sp_allocate_sparsity(fake, fake, 4, 0.5, 0.0, 0, 0.95, fake, fake, None) == 1
    assert lib.sp_allocate_sparsity(fake, fake, 0, 0.5, 1.0, 0, 0.95, fake, fake, None) == 2
    assert lib.sp_allocate_sparsity(fake, fake, 4, 0.5, 1.0, 7, 0.95, fake, fake, None) == 9
    # sp_gram_accumulate: dtype and shape checks
    x = api.SpMat(0x1000, api.SP_F64, 0, 8, 16, 16)
    assert lib.sp_gram_accumulate(C.byref(x), None, fake, 16, None, 0, None, None, None, 0, None) == 3
    x = api.SpMat(0x1000, api.SP_F32, 0, 8, 16, 8)
    assert lib.sp_gram_accumulate(C.byref(x), None, fake, 16, None, 0, None, None, None, 0, None) == 2
    # sp_ridge_solve: workspace too small
    assert lib.sp_ridge_solve(fake, 8, fake, 8, 4, 8, 0.1, 1, 1, fake, 8, None, fake, 16, None) == 5
    # a workspace that is large enough but not 256-byte aligned is refused before any launch
    need = api.workspace_bytes(api.SP_WS_RIDGE_SOLVE, 4, 8, 0, 0, api.SP_F64)
    assert lib.sp_ridge_solve(fake, 8, fake, 8, 4, 8, 0.1, 1, 1, fake, 8, None, C.c_void_p(0x1008), need, None) == 4
    need = api.workspace_bytes(api.SP_WS_LINEAR_REFIT, 4, 8, 0, 0, api.SP_F64)
    assert lib.sp_linear_refit(fake, 8, fake, 8, 4, 8, 1, fake, 4, 0.1, 1, 1, fake, 8, None, C.c_void_p(0x1010), need,
                               None) == 4
    # sp_admm_step: null params
    assert lib.sp_admm_step(None, None, None, None, None, None, 0, None) == 1


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(RuntimeError):
        api.sp_symmetrize(torch.zeros(4, 4))
