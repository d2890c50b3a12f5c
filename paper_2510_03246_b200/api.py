"""Thin ctypes binding over libsp.so (argument marshalling and buffer allocation only).

Every function here has the name of the C entry point it forwards to (see include/sp.h); all arithmetic runs in the
CUDA library.  PyTorch supplies device memory and the current stream.  There is no CPU fallback: if libsp.so is
missing or a CUDA device is absent the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsp.so")

SP_OK = 0
SP_F32, SP_BF16, SP_F64 = 0, 1, 2
SP_ACT_RELU, SP_ACT_SWIGLU = 0, 1
SP_Z_PAPER, SP_Z_EXACT = 0, 1
SP_SCORE_WANDA_L2, SP_SCORE_WANDA_L1, SP_SCORE_LEMMA1 = 0, 1, 2
SP_ALLOC_SOFTMAX, SP_ALLOC_INVERSE, SP_ALLOC_UNIFORM = 0, 1, 2
(SP_WS_GRAM, SP_WS_ADMM_STEP, SP_WS_SCORES, SP_WS_APPLY_MASK, SP_WS_FFN_INIT, SP_WS_LINEAR_REFIT, SP_WS_GEMM,
 SP_WS_RIDGE_SOLVE) = range(8)

EXPORTS = ["sp_gram_accumulate", "sp_ffn_init", "sp_admm_step", "sp_admm_scores", "sp_struct_scores",
           "sp_allocate_sparsity",
           "sp_apply_mask", "sp_apply_mask_batched", "sp_weight_stats", "sp_distribute_importance",
           "sp_struct_scores_static", "sp_ridge_solve", "sp_linear_refit", "sp_gemm", "sp_symmetrize", "sp_workspace_bytes", "sp_admm_overlap_bytes",
           "sp_status_string", "sp_version", "sp_profile_begin", "sp_profile_read", "sp_profile_kinds",
           "sp_profile_kind_name", "sp_launch_count", "sp_mha_init", "sp_mha_step", "sp_mha_workspace_bytes",
           "sp_set_reproducible", "sp_get_reproducible", "sp_allocate_sparsity_grid", "sp_apply_mask_global",
           "sp_apply_mask_global_bytes", "sp_objective_accumulate", "sp_ffn_cache_input_inverse",
           "sp_set_wait_budget", "sp_mha_value_refit", "sp_mha_value_refit_workspace_bytes"]


class SpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (sp_status {code})")


class SpMat(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("reserved", C.c_int32), ("rows", C.c_int64),
                ("cols", C.c_int64), ("ld", C.c_int64)]


class SpFfnModule(C.Structure):
    _fields_ = [("X", SpMat), ("Ypre", SpMat), ("W1_0", SpMat), ("W2_0", SpMat), ("d", C.c_int64), ("n", C.c_int64),
                ("N", C.c_int64), ("act", C.c_int32), ("reserved", C.c_int32), ("Wg_0", SpMat)]


class SpFfnState(C.Structure):
    _fields_ = [("Z", C.c_void_p), ("U", C.c_void_p), ("G_X", C.c_void_p), ("G_A", C.c_void_p), ("R1", C.c_void_p),
                ("R2", C.c_void_p), ("absA", C.c_void_p), ("W1", C.c_void_p), ("W2", C.c_void_p),
                ("scores", C.c_void_p), ("mask", C.c_void_p), ("importance", C.c_void_p), ("Gate", C.c_void_p),
                ("G_X_inv", C.c_void_p), ("G_A_perm", C.c_void_p), ("R2_perm", C.c_void_p), ("decay_tag", C.c_void_p),
                ("R1_perm", C.c_void_p), ("H_next", C.c_void_p), ("H_next_ld", C.c_int64)]


class SpAdmmParams(C.Structure):
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double), ("rho", C.c_double), ("rho_relative", C.c_int32),
                ("z_rule", C.c_int32), ("dual_mode", C.c_int32), ("score_kind", C.c_int32), ("k_keep", C.c_int64),
                ("reselect_mask", C.c_int32), ("refit", C.c_int32), ("token_chunk", C.c_int64),
                ("compute_objective", C.c_int32), ("skip_scores", C.c_int32)]


class SpScoreInputs(C.Structure):
    _fields_ = [("W", SpMat), ("colsq", C.c_void_p), ("colsq_stride", C.c_int64), ("colabs", C.c_void_p),
                ("inv_tokens", C.c_double), ("b", SpMat), ("c", SpMat), ("dd", SpMat), ("t", SpMat)]


class SpMhaModule(C.Structure):
    _fields_ = [("X", SpMat), ("Ypre", SpMat), ("Wq", SpMat), ("Wk", SpMat), ("Wv", SpMat), ("Wo", SpMat),
                ("d", C.c_int64), ("n_heads", C.c_int64), ("T", C.c_int64), ("n_seq", C.c_int64)]


class SpMhaState(C.Structure):
    _fields_ = [("Zq", C.c_void_p), ("Zk", C.c_void_p), ("P", C.c_void_p), ("Aattn", C.c_void_p),
                ("G_X", C.c_void_p), ("R_Q", C.c_void_p), ("R_K", C.c_void_p), ("G_attn", C.c_void_p),
                ("R_O", C.c_void_p)]


class SpMhaParams(C.Structure):
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double), ("a_steps", C.c_int32), ("z_steps", C.c_int32),
                ("eta_z", C.c_double), ("causal", C.c_int32), ("reserved", C.c_int32), ("seq_chunk", C.c_int64)]


REPORT_FIELDS = ["res_act", "res_out", "res_in", "z_sq", "a_sq", "rho1_eff", "rho2_eff", "kept", "factor_reused",
                 "pruned_scaled"]

_lib = None


def lib() -> C.CDLL:
    """Load libsp.so (built in-tree by paper_2510_03246_b200/build.py); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2510_03246_b200.build` first")
        L = C.CDLL(LIB_PATH)
        L.sp_workspace_bytes.restype = C.c_size_t
        L.sp_workspace_bytes.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_int32]
        L.sp_admm_overlap_bytes.restype = C.c_size_t
        L.sp_admm_overlap_bytes.argtypes = [C.c_int64, C.c_int64]
        L.sp_status_string.restype = C.c_char_p
        L.sp_status_string.argtypes = [C.c_int32]
        L.sp_version.restype = C.c_int32
        vp, i32, i64, dbl, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_double, C.c_size_t
        pm = C.POINTER(SpMat)
        L.sp_gram_accumulate.argtypes = [pm, pm, vp, i64, vp, i64, vp, vp, vp, sz, vp]
        L.sp_ffn_init.argtypes = [C.POINTER(SpFfnModule), C.POINTER(SpFfnState), i64, vp, vp, sz, vp]
        L.sp_ffn_cache_input_inverse.argtypes = [C.POINTER(SpFfnModule), C.POINTER(SpFfnState), dbl, i32, vp, vp, sz, vp]
        L.sp_admm_scores.argtypes = [C.POINTER(SpFfnModule), C.POINTER(SpFfnState), C.POINTER(SpAdmmParams), vp, vp,
                                     C.c_size_t, vp]
        L.sp_admm_step.argtypes = [C.POINTER(SpFfnModule), C.POINTER(SpFfnState), C.POINTER(SpAdmmParams), vp, vp, vp,
                                   sz, vp]
        L.sp_struct_scores.argtypes = [i32, i32, C.POINTER(SpScoreInputs), i64, vp, vp, vp, dbl, vp, sz, vp]
        L.sp_struct_scores_static.argtypes = [i32, i32, C.POINTER(SpScoreInputs), i64, vp, vp, vp]
        L.sp_allocate_sparsity.argtypes = [vp, vp, i32, dbl, dbl, i32, dbl, vp, vp, vp]
        L.sp_apply_mask.argtypes = [vp, i64, i64, i32, vp, vp, vp, pm, pm, vp, sz, vp]
        L.sp_apply_mask_batched.argtypes = [vp, i64, i64, i32, vp, vp, i64, vp, vp, i64, vp]
        L.sp_weight_stats.argtypes = [pm, i32, i64, i32, vp, vp, sz, vp]
        L.sp_distribute_importance.argtypes = [vp, i32, vp, i32, i32, dbl, dbl, vp, vp, vp]
        L.sp_ridge_solve.argtypes = [vp, i64, vp, i64, i64, i64, dbl, i32, i32, vp, i64, vp, vp, sz, vp]
        L.sp_linear_refit.argtypes = [vp, i64, vp, i64, i64, i64, i32, vp, i64, dbl, i32, i32, vp, i64, vp, vp, sz, vp]
        L.sp_gemm.argtypes = [i32, i32, i64, i64, i64, dbl, pm, pm, dbl, pm, i32, i32, vp, vp]
        L.sp_symmetrize.argtypes = [vp, i64, i64, vp]
        L.sp_mha_workspace_bytes.restype = C.c_size_t
        L.sp_mha_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, i32]
        L.sp_mha_init.argtypes = [C.POINTER(SpMhaModule), C.POINTER(SpMhaState), i32, i64, vp, vp, sz, vp]
        L.sp_mha_step.argtypes = [C.POINTER(SpMhaModule), C.POINTER(SpMhaState), C.POINTER(SpMhaParams), vp, vp, sz, vp]
        L.sp_mha_value_refit_workspace_bytes.restype = C.c_size_t
        L.sp_mha_value_refit_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, i32]
        L.sp_mha_value_refit.argtypes = [C.POINTER(SpMhaModule), C.POINTER(SpMhaState), vp, dbl, i32, i64, vp, i64, vp, vp,
                                         sz, vp]
        L.sp_allocate_sparsity_grid.argtypes = [vp, vp, i32, dbl, vp, i32, i32, i32, dbl, vp, vp, vp]
        L.sp_apply_mask_global.argtypes = [vp, i64, i64, i32, dbl, i64, vp, i64, vp, vp, vp, sz, vp]
        L.sp_apply_mask_global_bytes.restype = C.c_size_t
        L.sp_apply_mask_global_bytes.argtypes = [i64, i32]
        L.sp_objective_accumulate.argtypes = [vp, dbl, vp, i32, vp]
        L.sp_set_reproducible.argtypes = [i32]
        L.sp_set_wait_budget.argtypes = [i64]
        L.sp_get_reproducible.restype = i32
        L.sp_profile_begin.argtypes = [i32]
        L.sp_profile_read.argtypes = [vp]
        L.sp_profile_kinds.restype = i32
        L.sp_profile_kind_name.restype = C.c_char_p
        L.sp_profile_kind_name.argtypes = [i32]
        L.sp_launch_count.restype = i64
        for name in EXPORTS:
            if name not in ("sp_workspace_bytes", "sp_admm_overlap_bytes", "sp_mha_workspace_bytes",
                            "sp_mha_value_refit_workspace_bytes",
                            "sp_apply_mask_global_bytes", "sp_status_string", "sp_version", "sp_profile_kinds",
                            "sp_profile_kind_name", "sp_launch_count"):
                getattr(L, name).restype = C.c_int32
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().sp_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != SP_OK:
        raise SpError(code, where)


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise RuntimeError("libsp operates on CUDA tensors only (there is no CPU path)")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dt(t: torch.Tensor) -> int:
    return {torch.float32: SP_F32, torch.bfloat16: SP_BF16, torch.float64: SP_F64}[t.dtype]


def mat(t: torch.Tensor | None) -> SpMat:
    """Row-major matrix view of a 2-D tensor whose last dimension is contiguous."""
    if t is None:
        return SpMat(None, 0, 0, 0, 0, 0)
    assert t.dim() == 2 and (t.stride(1) == 1 or t.shape[1] <= 1), "need a row-major 2-D tensor"
    return SpMat(t.data_ptr(), _dt(t), 0, t.shape[0], t.shape[1], t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0)))


def _ptr(t: torch.Tensor | None):
    return None if t is None else t.data_ptr()


def workspace_bytes(op: int, d: int, n: int, N: int, token_chunk: int = 0, dtype: int = SP_F32) -> int:
    return int(lib().sp_workspace_bytes(op, d, n, N, token_chunk, dtype))


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(4, dtype=torch.int32, device=device)


def sp_set_reproducible(on: bool):
    """Process-wide switch: fixed summation order everywhere (bit-identical results for equal inputs)."""
    _check(lib().sp_set_reproducible(int(bool(on))), "sp_set_reproducible")


def sp_profile_begin(enable=True):
    """0 / False: off; 1 / True: outermost kernels and phases; 2: every kernel, also inside a phase."""
    _check(lib().sp_profile_begin(int(enable)), "sp_profile_begin")


def sp_profile_read() -> dict:
    """Per kernel kind: records, total ms, algorithmic flops and bytes (call after synchronising the stream)."""
    L = lib()
    nk = L.sp_profile_kinds()
    buf = (C.c_double * (nk * 4))()
    _check(L.sp_profile_read(buf), "sp_profile_read")
    out = {}
    for k in range(nk):
        name = L.sp_profile_kind_name(k).decode()
        out[name] = dict(records=int(buf[k * 4]), ms=buf[k * 4 + 1], flops=buf[k * 4 + 2], bytes=buf[k * 4 + 3])
    return out


def sp_launch_count() -> int:
    return int(lib().sp_launch_count())


# ---------------------------------------------------------------------------------------------- direct calls
def sp_gemm(A, B, C_, transA=False, transB=False, alpha=1.0, beta=0.0, lower_only=False, use_tensor_cores=False,
            status=None, M=None, N=None, K=None):
    """C = alpha * op(A) op(B) + beta * C."""
    _require_cuda(A, B, C_)
    M = C_.shape[0] if M is None else M
    N = C_.shape[1] if N is None else N
    K = (A.shape[0] if transA else A.shape[1]) if K is None else K
    a, b, c = mat(A), mat(B), mat(C_)
    _check(lib().sp_gemm(int(transA), int(transB), M, N, K, alpha, C.byref(a), C.byref(b), beta, C.byref(c),
                         int(lower_only), int(use_tensor_cores), _ptr(status), _stream()), "sp_gemm")


def sp_symmetrize(G):
    _require_cuda(G)
    _check(lib().sp_symmetrize(G.data_ptr(), G.shape[0], G.stride(0), _stream()), "sp_symmetrize")


def sp_gram_accumulate(Xc, Yc, G, R=None, rowstats=None, status=None, ws=None):
    _require_cuda(Xc, Yc, G, R, rowstats)
    x = mat(Xc)
    y = mat(Yc) if Yc is not None else None
    if ws is None:
        ws = _ws(workspace_bytes(SP_WS_GRAM, Xc.shape[1], 0, Xc.shape[0], 0, _dt(Xc)), Xc.device)
    _check(lib().sp_gram_accumulate(C.byref(x), C.byref(y) if y is not None else None, G.data_ptr(), G.stride(0),
                                    _ptr(R), R.stride(0) if R is not None else 0, _ptr(rowstats), _ptr(status),
                                    ws.data_ptr(), ws.numel(), _stream()), "sp_gram_accumulate")


def sp_ridge_solve(R, G, rho, rho_relative=True, precise=False, W=None, status=None, ws=None):
    _require_cuda(R, G, W)
    m, n = R.shape
    if W is None:
        W = torch.empty_like(R)
    if ws is None:
        ws = _ws(workspace_bytes(SP_WS_RIDGE_SOLVE, m, n, 0, 0, SP_F64 if precise else SP_F32), R.device)
    _check(lib().sp_ridge_solve(R.data_ptr(), R.stride(0), G.data_ptr(), G.stride(0), m, n, float(rho),
                                int(rho_relative), int(precise), W.data_ptr(), W.stride(0), _ptr(status),
                                ws.data_ptr(), ws.numel(), _stream()), "sp_ridge_solve")
    return W


def sp_linear_refit(R, G, mask, k_keep, rho, group=1, precise=False, W=None, status=None, ws=None,
                    rho_relative=False):
    _require_cuda(R, G, mask, W)
    m, n = R.shape
    if W is None:
        W = torch.empty_like(R)
    if ws is None:
        ws = _ws(workspace_bytes(SP_WS_LINEAR_REFIT, m, n, 0, 0, SP_F64 if precise else SP_F32), R.device)
    _check(lib().sp_linear_refit(R.data_ptr(), R.stride(0), G.data_ptr(), G.stride(0), m, n // group, group,
                                 mask.data_ptr(), int(k_keep), float(rho), int(rho_relative), int(precise), W.data_ptr(),
                                 W.stride(0), _ptr(status), ws.data_ptr(), ws.numel(), _stream()), "sp_linear_refit")
    return W


def sp_struct_scores(kind, n_units, group=1, W=None, colsq=None, colsq_stride=1, colabs=None, inv_tokens=0.0,
                     b=None, c=None, dd=None, t=None, r_layer=0.0, want_relaxed=False, ws=None):
    """Returns (scores fp32 [n_units], importance fp64 [1], relaxed fp64 [n_units] or None)."""
    dev = (W if W is not None else b).device
    _require_cuda(W, colsq, colabs, b, c, dd, t)
    inp = SpScoreInputs(mat(W), _ptr(colsq), colsq_stride, _ptr(colabs), float(inv_tokens), mat(b), mat(c), mat(dd),
                        mat(t))
    scores = torch.empty(n_units, dtype=torch.float32, device=dev)
    imp = torch.empty(1, dtype=torch.float64, device=dev)
    relaxed = torch.empty(n_units, dtype=torch.float64, device=dev) if want_relaxed else None
    rows = W.shape[0] if W is not None else b.shape[0]
    if ws is None:
        ws = _ws(workspace_bytes(SP_WS_SCORES, n_units * group, 0, rows, 0, SP_F32), dev)
    _check(lib().sp_struct_scores(kind, group, C.byref(inp), n_units, scores.data_ptr(), imp.data_ptr(),
                                  _ptr(relaxed), float(r_layer), ws.data_ptr(), ws.numel(), _stream()),
           "sp_struct_scores")
    return scores, imp, relaxed


STATIC_SCORES_MAX_COLS = 32768


def sp_struct_scores_static(kind, n_units, scores, importance, group=1, W=None, colsq=None, colsq_stride=1,
                            colabs=None, inv_tokens=0.0):
    """Wanda scores without a workspace: for callers that cannot allocate device memory at the time of the call.

    `scores` (fp32 [n_units]) and `importance` (fp64 [1]) are caller-provided outputs; nothing is allocated here or in
    the library.  Sizes beyond the built-in scratch raise SpError (SP_ERR_STATIC_LIMIT)."""
    _require_cuda(W, colsq, colabs, scores, importance)
    inp = SpScoreInputs(mat(W), _ptr(colsq), colsq_stride, _ptr(colabs), float(inv_tokens), mat(None), mat(None),
                        mat(None), mat(None))
    _check(lib().sp_struct_scores_static(kind, group, C.byref(inp), n_units, scores.data_ptr(), _ptr(importance),
                                         _stream()), "sp_struct_scores_static")


def sp_allocate_sparsity(I, n_units, rbar, T, mode=SP_ALLOC_SOFTMAX, clip_hi=0.95):
    """I: fp64 [L] device, n_units: int64 [L] device.  Returns (r fp64 [L], k_keep int64 [L])."""
    _require_cuda(I, n_units)
    L = I.numel()
    r = torch.empty(L, dtype=torch.float64, device=I.device)
    k = torch.empty(L, dtype=torch.int64, device=I.device)
    _check(lib().sp_allocate_sparsity(I.data_ptr(), n_units.data_ptr(), L, float(rbar), float(T), mode,
                                      float(clip_hi), r.data_ptr(), k.data_ptr(), _stream()), "sp_allocate_sparsity")
    return r, k


def sp_allocate_sparsity_grid(I, n_units, rbar, T_list, T_relative=True, mode=SP_ALLOC_SOFTMAX, clip_hi=0.95):
    """Allocation for every temperature of T_list (fp64 [n_T] device) in one launch.  Returns (r [n_T, L], k_keep)."""
    _require_cuda(I, n_units, T_list)
    L, nT = I.numel(), T_list.numel()
    r = torch.empty(nT, L, dtype=torch.float64, device=I.device)
    k = torch.empty(nT, L, dtype=torch.int64, device=I.device)
    _check(lib().sp_allocate_sparsity_grid(I.data_ptr(), n_units.data_ptr(), L, float(rbar), T_list.data_ptr(), nT,
                                           int(bool(T_relative)), mode, float(clip_hi), r.data_ptr(), k.data_ptr(),
                                           _stream()), "sp_allocate_sparsity_grid")
    return r, k


def sp_apply_mask_global(scores, keep_fraction, min_keep=0, mask_out=None):
    """scores: fp32 [L, n] (rows contiguous).  Returns (mask u8 [L, n], tau fp32 [1], kept int64 [L])."""
    _require_cuda(scores, mask_out)
    L, n = scores.shape
    mask = mask_out if mask_out is not None else torch.empty(L, n, dtype=torch.uint8, device=scores.device)
    tau = torch.empty(1, dtype=torch.float32, device=scores.device)
    kept = torch.empty(L, dtype=torch.int64, device=scores.device)
    ws = _ws(lib().sp_apply_mask_global_bytes(n, L), scores.device)
    _check(lib().sp_apply_mask_global(scores.data_ptr(), scores.stride(0), n, L, float(keep_fraction), int(min_keep),
                                      mask.data_ptr(), mask.stride(0), tau.data_ptr(), kept.data_ptr(), ws.data_ptr(),
                                      ws.numel(), _stream()), "sp_apply_mask_global")
    return mask, tau, kept


def sp_objective_accumulate(report, beta, loss, accumulate=True):
    """loss[0] (+)= objective of the step report (device tensors)."""
    _require_cuda(report, loss)
    _check(lib().sp_objective_accumulate(report.data_ptr(), float(beta), loss.data_ptr(), int(bool(accumulate)),
                                         _stream()), "sp_objective_accumulate")


def sp_apply_mask(scores, k_keep, group=1, W_rows=None, W_cols=None, want_index=False, mask_out=None):
    """Returns (mask u8 [n_units], tau fp32 [1], kept_idx int32 [k_keep] or None); W_rows / W_cols are zeroed in place.
    mask_out: caller-owned contiguous uint8 [n_units] buffer to write the mask into."""
    _require_cuda(scores, W_rows, W_cols, mask_out)
    n = scores.numel()
    if mask_out is not None and (mask_out.dtype != torch.uint8 or mask_out.numel() != n or not mask_out.is_contiguous()):
        raise ValueError("mask_out must be contiguous uint8 [n_units]")
    if not scores.is_contiguous() or scores.dtype != torch.float32:
        raise ValueError("scores must be contiguous fp32")
    mask = mask_out if mask_out is not None else torch.empty(n, dtype=torch.uint8, device=scores.device)
    tau = torch.empty(1, dtype=torch.float32, device=scores.device)
    idx = torch.empty(max(int(k_keep), 1), dtype=torch.int32, device=scores.device) if want_index else None
    wr = mat(W_rows) if W_rows is not None else None
    wc = mat(W_cols) if W_cols is not None else None
    _check(lib().sp_apply_mask(scores.data_ptr(), n, int(k_keep), group, mask.data_ptr(), tau.data_ptr(), _ptr(idx),
                               C.byref(wr) if wr is not None else None, C.byref(wc) if wc is not None else None,
                               None, 0, _stream()), "sp_apply_mask")
    return mask, tau, (idx[:int(k_keep)] if idx is not None else None)


def sp_apply_mask_batched(scores, k_keep, want_index=False):
    """Top-k selection of all layers in one launch.  scores fp32 [L, n_units]; k_keep int64 [L] on the device.
    Returns (mask u8 [L, n_units], tau fp32 [L], kept_idx int32 [L, n_units] or None; row l holds k_keep[l] entries)."""
    _require_cuda(scores, k_keep)
    if scores.dim() != 2 or scores.dtype != torch.float32 or scores.stride(1) != 1:
        raise ValueError("scores must be fp32 [L, n_units] with unit inner stride")
    if k_keep.dtype != torch.int64 or k_keep.numel() != scores.shape[0] or not k_keep.is_contiguous():
        raise ValueError("k_keep must be contiguous int64 [L]")
    L, n = scores.shape
    mask = torch.empty(L, n, dtype=torch.uint8, device=scores.device)
    tau = torch.empty(L, dtype=torch.float32, device=scores.device)
    idx = torch.full((L, n), -1, dtype=torch.int32, device=scores.device) if want_index else None
    _check(lib().sp_apply_mask_batched(scores.data_ptr(), scores.stride(0), n, L, k_keep.data_ptr(), mask.data_ptr(), n,
                                       tau.data_ptr(), _ptr(idx), n, _stream()), "sp_apply_mask_batched")
    return mask, tau, idx


SP_WS_WEIGHT_STATS = 8
SP_WS_INPUT_INVERSE = 9


def sp_weight_stats(W, axis=0, group=0, stats=None, accumulate=False):
    """Sums {|w|, w, w^2, count} over row blocks (axis 0) or column blocks (axis 1) of `group` rows / columns of W
    (group 0: the whole matrix).  Returns stats fp64 [n_blocks, 4]; with accumulate the sums are added to `stats`."""
    _require_cuda(W, stats)
    rows, cols = W.shape
    nb = 1 if group == 0 else (rows // group if axis == 0 else cols // group)
    if stats is None:
        stats = torch.zeros(nb, 4, dtype=torch.float64, device=W.device)
        accumulate = False
    ws = _ws(workspace_bytes(SP_WS_WEIGHT_STATS, nb, 0, 0), W.device)
    m = mat(W)
    _check(lib().sp_weight_stats(C.byref(m), axis, group, int(accumulate), stats.data_ptr(), ws.data_ptr(), ws.numel(),
                                 _stream()), "sp_weight_stats")
    return stats


def sp_distribute_importance(head_stats, fc_stats, rho, gamma):
    """head_stats fp64 [L, H, 4] or None, fc_stats fp64 [L, n_fc, 4] or None.  Returns (I_attn [L] or None, I_mlp)."""
    ref = head_stats if head_stats is not None else fc_stats
    _require_cuda(head_stats, fc_stats)
    L = ref.shape[0]
    Ia = torch.empty(L, dtype=torch.float64, device=ref.device) if head_stats is not None else None
    Im = torch.empty(L, dtype=torch.float64, device=ref.device) if fc_stats is not None else None
    _check(lib().sp_distribute_importance(_ptr(head_stats), head_stats.shape[1] if head_stats is not None else 0,
                                          _ptr(fc_stats), fc_stats.shape[1] if fc_stats is not None else 0, L,
                                          float(rho), float(gamma), _ptr(Ia), _ptr(Im), _stream()),
           "sp_distribute_importance")
    return Ia, Im


# ---------------------------------------------------------------------------------------------- module driver
@dataclass
class AdmmParams:
    alpha: float = 1.0
    beta: float = 1.0
    rho: float = 0.1
    rho_relative: bool = True
    z_rule: int = SP_Z_PAPER
    dual_mode: bool = False
    score_kind: int = SP_SCORE_WANDA_L2
    k_keep: int = 0
    reselect_mask: bool = True
    refit: bool = True
    token_chunk: int = 0
    compute_objective: bool = False
    skip_scores: bool = False       # fixed mask (reselect_mask False, refit True): skip W2~ and the scores

    def to_c(self) -> SpAdmmParams:
        return SpAdmmParams(self.alpha, self.beta, self.rho, int(self.rho_relative), self.z_rule, int(self.dual_mode),
                            self.score_kind, int(self.k_keep), int(self.reselect_mask), int(self.refit),
                            int(self.token_chunk), int(self.compute_objective), int(self.skip_scores))


class FfnModule:
    """Owns the device buffers of one FFN module and forwards to sp_ffn_init / sp_admm_step."""
    report_fields = REPORT_FIELDS

    def __init__(self, X: torch.Tensor, W1_0: torch.Tensor, W2_0: torch.Tensor, dual_mode: bool = False,
                 token_chunk: int = 0, overlap_k: int = 0, Wg_0: torch.Tensor | None = None,
                 scores: torch.Tensor | None = None, mask: torch.Tensor | None = None, ws_pool: dict | None = None,
                 pruned_decay: bool = True):
        """overlap_k > 0: also reserve the optional workspace tail that lets sp_admm_step compute z1 of all tokens
        beside the kept-support recovery, sized for overlap_k kept units (see sp_admm_overlap_bytes).
        Wg_0 (gate projection [n, d]) makes the module a SwiGLU one: W1_0 is then its up projection.
        scores (fp32 [n]) / mask (uint8 [n]): caller-owned contiguous buffers, e.g. rows of one [L, n] array over
        which a lock-step run selects a single global threshold.  ws_pool: a dict shared by modules that are never
        in flight at the same time; they then use one workspace.
        pruned_decay (bf16 storage, ReLU, no dual variable): hold the ordered accumulators of sp_ffn_state (G_A_perm,
        R2_perm, decay_tag; with overlap_k > 0 also R1_perm and H_next, sized for overlap_k kept units), with which a
        step whose mask stays scales the pruned channels' parts of G_A, R1, R2 instead of contracting them again.
        Code that writes Z of such a module itself must set decay_tag[1] = -1 afterwards."""
        _require_cuda(X, W1_0, W2_0, Wg_0)
        assert X.dtype in (torch.float32, torch.bfloat16)
        self.X = X.contiguous()
        self.N, self.d = X.shape
        self.n = W1_0.shape[0]
        dev = X.device
        self.dev = dev
        self.W1_0 = W1_0.to(torch.float32).contiguous()
        self.W2_0 = W2_0.to(torch.float32).contiguous()
        self.Wg_0 = Wg_0.to(torch.float32).contiguous() if Wg_0 is not None else None
        self.act = SP_ACT_SWIGLU if Wg_0 is not None else SP_ACT_RELU
        N, d, n = self.N, self.d, self.n
        f32 = dict(dtype=torch.float32, device=dev)
        self.Gate = torch.empty(N, n, **f32) if Wg_0 is not None else None
        self.Ypre = torch.empty(N, d, dtype=X.dtype, device=dev)
        self.Z = torch.empty(N, n, **f32)
        self.U = torch.zeros(N, n, **f32) if dual_mode else None
        self.G_X = torch.empty(d, d, **f32)
        self.G_X_inv = None           # cache of (G_X + rho1 I)^-1, see sp_ffn_cache_input_inverse
        self._inv_key = None
        self.cache_input_inverse = X.dtype == torch.bfloat16
        self.G_A = torch.empty(n, n, **f32)
        self.R1 = torch.empty(n, d, **f32)
        self.R2 = torch.empty(d, n, **f32)
        self.absA = torch.empty(n, dtype=torch.float64, device=dev)
        self.W1 = torch.zeros(n, d, **f32)
        self.W2 = torch.zeros(d, n, **f32)
        if scores is not None:
            assert scores.dtype == torch.float32 and scores.shape == (n,) and scores.is_contiguous() and scores.is_cuda
        if mask is not None:
            assert mask.dtype == torch.uint8 and mask.shape == (n,) and mask.is_contiguous() and mask.is_cuda
        self.scores = scores if scores is not None else torch.zeros(n, **f32)
        self.mask = mask if mask is not None else torch.ones(n, dtype=torch.uint8, device=dev)
        self.importance = torch.zeros(1, dtype=torch.float64, device=dev)
        self.report = torch.zeros(len(REPORT_FIELDS), dtype=torch.float64, device=dev)
        self.status = new_status(dev)
        self.token_chunk = token_chunk
        self.overlap_k = int(overlap_k)
        # ordered accumulators that let a step scale, instead of recompute, the parts of G_A and R2 that belong to
        # pruned channels while the mask stays (see sp_ffn_state.G_A_perm); ReLU modules without the dual variable
        self.G_A_perm = self.R2_perm = self.decay_tag = self.R1_perm = self.H_next = None
        if pruned_decay and X.dtype == torch.bfloat16 and Wg_0 is None and not dual_mode and n % 4 == 0:
            self.G_A_perm = torch.empty(n, n, **f32)
            self.R2_perm = torch.empty(d, n, **f32)
            self.decay_tag = torch.full((n + 8,), -1, dtype=torch.int32, device=dev)
            if overlap_k > 0:        # sized for that many kept units, like the other optional buffers
                self.R1_perm = torch.empty(n, d, **f32)
                self.H_next = torch.empty(N, (int(overlap_k) + 7) // 8 * 8, dtype=torch.bfloat16, device=dev)
        self._pool = ws_pool if ws_pool is not None else {}
        self.iteration = 0

    def h_next_rows(self, k: int, token_chunk: int) -> torch.Tensor:
        """[N, k] view-by-copy of the h that the last step left for the next one in H_next (sp_ffn_state.H_next: per
        token chunk a [k, Tc] block, tokens contiguous, at element t0 * H_next_ld)."""
        flat, ld = self.H_next.view(-1), self.H_next.shape[1]
        chunk = int(token_chunk) if token_chunk else self.N
        out = []
        for t0 in range(0, self.N, chunk):
            Tc = min(chunk, self.N - t0)
            out.append(flat[t0 * ld: t0 * ld + k * Tc].view(k, Tc).t())
        return torch.cat(out, 0)

    @property
    def _ws(self):
        return self._pool.get("ws")

    @_ws.setter
    def _ws(self, t):
        self._pool["ws"] = t

    def _module(self) -> SpFfnModule:
        return SpFfnModule(mat(self.X), mat(self.Ypre), mat(self.W1_0), mat(self.W2_0), self.d, self.n, self.N,
                           self.act, 0, mat(self.Wg_0))

    def _state(self) -> SpFfnState:
        return SpFfnState(self.Z.data_ptr(), _ptr(self.U), self.G_X.data_ptr(), self.G_A.data_ptr(),
                          self.R1.data_ptr(), self.R2.data_ptr(), self.absA.data_ptr(), self.W1.data_ptr(),
                          self.W2.data_ptr(), self.scores.data_ptr(), self.mask.data_ptr(),
                          self.importance.data_ptr(), _ptr(self.Gate), _ptr(self.G_X_inv), _ptr(self.G_A_perm),
                          _ptr(self.R2_perm), _ptr(self.decay_tag), _ptr(self.R1_perm), _ptr(self.H_next),
                          self.H_next.shape[1] if self.H_next is not None else 0)

    def _workspace(self, chunk: int) -> torch.Tensor:
        need = max(workspace_bytes(SP_WS_ADMM_STEP, self.d, self.n, self.N, chunk, _dt(self.X)),
                   workspace_bytes(SP_WS_FFN_INIT, self.d, self.n, self.N, chunk, _dt(self.X)))
        if self.overlap_k > 0:
            need += int(lib().sp_admm_overlap_bytes(self.N, self.overlap_k))
        if self._ws is None or self._ws.numel() < need:
            self._ws = _ws(need, self.dev)
        return self._ws

    def sp_ffn_init(self):
        self._inv_key = None            # G_X is about to change
        ws = self._workspace(self.token_chunk)
        m, st = self._module(), self._state()
        _check(lib().sp_ffn_init(C.byref(m), C.byref(st), self.token_chunk, self.status.data_ptr(), ws.data_ptr(),
                                 ws.numel(), _stream()), "sp_ffn_init")
        self.iteration = 0

    def sp_ffn_cache_input_inverse(self, rho: float, rho_relative: bool = True):
        """(G_X + rho1 I)^-1 of the constant module input into self.G_X_inv (once per module and ridge)."""
        if self.G_X_inv is None:
            self.G_X_inv = torch.empty(self.d, self.d, dtype=torch.float32, device=self.dev)
        ws = _ws(workspace_bytes(SP_WS_INPUT_INVERSE, self.d, 0, 0, 0, 0), self.dev)
        m, st = self._module(), self._state()
        _check(lib().sp_ffn_cache_input_inverse(C.byref(m), C.byref(st), float(rho), int(bool(rho_relative)),
                                                self.status.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
               "sp_ffn_cache_input_inverse")
        self._inv_key = (float(rho), bool(rho_relative))

    def _ensure_inverse(self, p):
        if self.cache_input_inverse and self._inv_key != (float(p.rho), bool(p.rho_relative)):
            self.sp_ffn_cache_input_inverse(p.rho, p.rho_relative)

    def sp_admm_step(self, p: AdmmParams):
        self._ensure_inverse(p)
        chunk = p.token_chunk or self.token_chunk
        ws = self._workspace(chunk)
        m, st = self._module(), self._state()
        cp = p.to_c()
        cp.token_chunk = chunk
        _check(lib().sp_admm_step(C.byref(m), C.byref(st), C.byref(cp), self.report.data_ptr(),
                                  self.status.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "sp_admm_step")
        self.iteration += 1

    def sp_admm_scores(self, p: AdmmParams):
        """Unrestricted recovery + unit scores + layer importance of the current state (no mask, no token pass)."""
        self._ensure_inverse(p)
        chunk = p.token_chunk or self.token_chunk
        ws = self._workspace(chunk)
        m, st = self._module(), self._state()
        cp = p.to_c()
        cp.token_chunk = chunk
        _check(lib().sp_admm_scores(C.byref(m), C.byref(st), C.byref(cp), self.status.data_ptr(), ws.data_ptr(),
                                    ws.numel(), _stream()), "sp_admm_scores")

    def select_mask(self, k_keep: int):
        """Top-k of the current scores into the module's mask (what a step does when it reselects)."""
        sp_apply_mask(self.scores, k_keep, mask_out=self.mask)

    def read_report(self) -> dict:
        return dict(zip(REPORT_FIELDS, self.report.cpu().tolist()))

    def check_status(self):
        s = self.status.cpu().tolist()
        if s[0] != 0:
            raise SpError(s[0], f"device status (index {s[1]}, aux {s[2]})")


@dataclass
class MhaParams:
    alpha: float = 1.0
    beta: float = 1.0
    a_steps: int = 4
    z_steps: int = 4
    eta_z: float = 1.0
    causal: bool = True
    seq_chunk: int = 0


class MhaModule:
    """Owns the device buffers of one attention module (Method 2 auxiliary variables) and forwards to sp_mha_init /
    sp_mha_step.  X: [n_seq * T, d] token-major; Wq, Wk, Wv, Wo: [d, d] ([out, in]), kept in fp32 for the library."""

    def __init__(self, X: torch.Tensor, Wq, Wk, Wv, Wo, n_heads: int, T: int, seq_chunk: int = 0,
                 accumulators: bool = True):
        _require_cuda(X, Wq, Wk, Wv, Wo)
        self.X = X.contiguous()
        self.dev = X.device
        N, d = X.shape
        assert N % T == 0 and d % n_heads == 0
        self.d, self.n_heads, self.T, self.n_seq, self.seq_chunk = d, n_heads, T, N // T, seq_chunk
        self.Wq, self.Wk, self.Wv, self.Wo = (w.float().contiguous() for w in (Wq, Wk, Wv, Wo))
        self.Ypre = torch.empty_like(self.X)
        f32 = dict(dtype=torch.float32, device=self.dev)
        self.Zq, self.Zk, self.Aattn = (torch.empty(N, d, **f32) for _ in range(3))
        self.P = torch.empty(self.n_seq, n_heads, T, T, **f32)
        # accumulators of the weight recoveries (rebuilt by every init / step)
        self.G_X, self.R_Q, self.R_K, self.G_attn, self.R_O = ((torch.empty(d, d, **f32) for _ in range(5))
                                                               if accumulators else (None,) * 5)
        self.status = new_status(self.dev)
        self._wsbuf = _ws(lib().sp_mha_workspace_bytes(d, n_heads, T, self.n_seq, seq_chunk, _dt(self.X)), self.dev)
        self._ws_refit = None       # workspace of sp_mha_value_refit, allocated on first use

    def set_weights(self, Wq, Wk, Wv, Wo):
        for dst, src in ((self.Wq, Wq), (self.Wk, Wk), (self.Wv, Wv), (self.Wo, Wo)):
            dst.copy_(src)

    def _module(self) -> SpMhaModule:
        return SpMhaModule(mat(self.X), mat(self.Ypre), mat(self.Wq), mat(self.Wk), mat(self.Wv), mat(self.Wo), self.d,
                           self.n_heads, self.T, self.n_seq)

    def _state(self) -> SpMhaState:
        return SpMhaState(self.Zq.data_ptr(), self.Zk.data_ptr(), self.P.data_ptr(), self.Aattn.data_ptr(),
                          _ptr(self.G_X), _ptr(self.R_Q), _ptr(self.R_K), _ptr(self.G_attn), _ptr(self.R_O))

    def sp_mha_init(self, causal: bool = True):
        m, st = self._module(), self._state()
        _check(lib().sp_mha_init(C.byref(m), C.byref(st), int(causal), self.seq_chunk, self.status.data_ptr(),
                                 self._wsbuf.data_ptr(), self._wsbuf.numel(), _stream()), "sp_mha_init")

    def sp_mha_step(self, p: MhaParams):
        m, st = self._module(), self._state()
        prm = SpMhaParams(p.alpha, p.beta, p.a_steps, p.z_steps, p.eta_z, int(p.causal), 0, self.seq_chunk)
        _check(lib().sp_mha_step(C.byref(m), C.byref(st), C.byref(prm), self.status.data_ptr(), self._wsbuf.data_ptr(),
                                 self._wsbuf.numel(), _stream()), "sp_mha_step")

    def sp_mha_value_refit(self, head_mask=None, rho: float = 0.0, rho_relative: bool = True,
                           out: torch.Tensor | None = None) -> torch.Tensor:
        """W_V recovered from the module's P and Aattn (see sp.h); head_mask: n_heads values on the HOST (None = all
        kept).  Writes into `out` (default: the module's own Wv) and returns it."""
        m, st = self._module(), self._state()
        out = self.Wv if out is None else out
        assert out.is_cuda and out.dtype == torch.float32 and out.shape == (self.d, self.d) and out.stride(1) == 1
        hm = None
        if head_mask is not None:
            hm = (C.c_uint8 * self.n_heads)(*[1 if int(v) else 0 for v in head_mask])
        need = lib().sp_mha_value_refit_workspace_bytes(self.d, self.n_heads, self.T, self.n_seq, self.seq_chunk,
                                                        _dt(self.X))
        if self._ws_refit is None or self._ws_refit.numel() < need:
            self._ws_refit = _ws(need, self.dev)
        _check(lib().sp_mha_value_refit(C.byref(m), C.byref(st), hm, float(rho), int(rho_relative), self.seq_chunk,
                                        out.data_ptr(), out.stride(0), self.status.data_ptr(),
                                        self._ws_refit.data_ptr(), self._ws_refit.numel(), _stream()),
               "sp_mha_value_refit")
        return out

    def check_status(self):
        code = int(self.status[0].item())
        if code != SP_OK:
            raise SpError(code, "device status")
