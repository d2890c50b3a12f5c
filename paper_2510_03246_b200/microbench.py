"""Per-kernel micro-benchmarks of libsp on one GPU (CUDA-event timings; also the small cases profiled with ncu).

    python -m paper_2510_03246_b200.microbench gemm  [--reps 5 --warm 2]   GEMM shapes of one C2 token chunk
    python -m paper_2510_03246_b200.microbench solve [--reps 3 --warm 1]   regularised solves of a C2 step

Inputs are random (torch.randn on the device): these runs time kernels, they check nothing.
"""
from __future__ import annotations

import argparse

import torch

from . import api

DEV = "cuda"
T, D, N = 16384, 2048, 8192      # tokens of one chunk, d_model, FFN channels of workload C2


def _timeit(fn, reps, warm):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def _rnd(shape, dt):
    return (torch.randn(*shape, device=DEV) * 0.5).to(dt)


def gemm_cases(reps, warm):
    bf, f32 = torch.bfloat16, torch.float32
    st = api.new_status()
    cases = [  # name, M, N, K, A K-major, B K-major, C dtype, beta, lower
        ("E = Ypre - H W2^T (bf16 out)", T, D, N // 2, True, True, bf, 1.0, False),
        ("D = E Q^T (f32 out)", T, N // 2, D, True, True, f32, 0.0, False),
        ("z1 = X [W1hi W1lo]^T (f32 out)", T, N // 2, 2 * D, True, True, f32, 0.0, False),
        ("G_A += A^T A (lower)", N, N, T, False, False, f32, 1.0, True),
        ("R2 += Ypre^T A", D, N, T, False, False, f32, 1.0, False),
        ("R1 += Z^T X", N, D, T, False, False, f32, 1.0, False),
        ("solve update (K = 6 x 128)", 2048, 4096, 768, True, True, f32, 1.0, False),
    ]
    for name, M, Nn, K, ak, bk, cdt, beta, lower in cases:
        A = _rnd((M, K) if ak else (K, M), bf)
        B = _rnd((Nn, K) if bk else (K, Nn), bf)
        C = _rnd((M, Nn), cdt)
        ms = _timeit(lambda: api.sp_gemm(A, B, C, transA=not ak, transB=bk, alpha=1.0, beta=beta, lower_only=lower,
                                         use_tensor_cores=True, status=st), reps, warm)
        fl = (1.0 if lower else 2.0) * M * Nn * K
        print(f"{name:34s} {M:6d} x {Nn:6d} x {K:6d}  {ms:8.3f} ms  {fl / ms / 1e9:8.1f} TFLOP/s", flush=True)
    print("status", st.cpu().tolist())


def solve_cases(reps, warm):
    st = api.new_status()
    for m, n in ((2048, 8192), (2048, 4096), (8192, 2048), (4096, 2048)):
        A = torch.relu(torch.randn(n, 2 * n, device=DEV))
        G = (A @ A.T).contiguous()
        R = torch.randn(m, n, device=DEV)
        W = torch.empty_like(R)
        ws = torch.empty(api.workspace_bytes(api.SP_WS_RIDGE_SOLVE, m, n, 0, 0, api.SP_F32), dtype=torch.uint8,
                         device=DEV)
        ms = _timeit(lambda: api.sp_ridge_solve(R, G, 0.1, True, False, W=W, status=st, ws=ws), reps, warm)
        api.sp_profile_begin(2)
        api.sp_ridge_solve(R, G, 0.1, True, False, W=W, status=st, ws=ws)
        torch.cuda.synchronize()
        pr = api.sp_profile_read()
        api.sp_profile_begin(0)
        fl = n ** 3 / 3 + 2.0 * m * n * n
        print(f"ridge solve m={m} n={n}: {ms:8.3f} ms  {fl / ms / 1e9:7.1f} TFLOP/s (algorithmic)")
        print("   " + "; ".join(f"{k}: {v['records']} x {1e3 * v['ms'] / max(v['records'], 1):.1f} us"
                                for k, v in pr.items() if v["records"]), flush=True)
    print("status", st.cpu().tolist())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["gemm", "solve"])
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--warm", type=int, default=2)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("microbench needs a CUDA device")
    api.lib()
    (gemm_cases if a.what == "gemm" else solve_cases)(a.reps, a.warm)


if __name__ == "__main__":
    main()
