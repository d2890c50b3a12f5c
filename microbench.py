"""Per-kernel micro-benchmarks of libsp on one GPU (CUDA-event timings; also the small cases profiled with ncu).

    python microbench.py gemm  [--reps 5 --warm 2]   GEMM shapes of one C2 token chunk
    python microbench.py solve [--reps 3 --warm 1]   regularised solves of a C2 step
    python microbench.py mask  [--reps 5 --warm 2]   scores, allocation and top-k as standalone
                                                                           kernels (L2 flushed before every call)
    python microbench.py mha   [--reps 3 --warm 1]   one outer step of the attention-module updates (Method 2):
                                                                           d = 2048, 32 heads, sequences of 1024 tokens
    python microbench.py lockstep [--reps 3 --warm 1] lock-step iterations of several C2-wide
                                                                           layers under one global threshold

Inputs are random (torch.randn on the device): these runs time kernels, they check nothing.
"""
from __future__ import annotations

import argparse

import torch

from paper_2510_03246_b200 import api

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
        # the accumulator products as a step issues them while the mask stays: the fused update leaves A channel-major
        # (K-major here) with the kept channels first, and only the kept columns are contracted anew
        ("G_A[:, kept] += A^T A_kept (lower)", N, N // 2, T, True, True, f32, 1.0, True),
        ("R2[:, kept] += Ypre^T A_kept", D, N // 2, T, False, True, f32, 1.0, False),
        ("R1[kept, :] += Z_kept^T X (Z^T K-major)", N // 2, D, T, True, False, f32, 1.0, False),
        ("solve update (K = 6 x 128)", 2048, 4096, 768, True, True, f32, 1.0, False),
        # the pruned parts, contracted only in a step whose mask changed
        ("G_A[pruned, pruned] (lower)", N // 2, N // 2, T, True, True, f32, 1.0, True),
        ("R2[:, pruned]", D, N // 2, T, False, True, f32, 1.0, False),
        ("R1[pruned, :]", N // 2, D, T, True, False, f32, 1.0, False),
        # the full products of a module without the ordered accumulators
        ("G_A += A^T A (lower, A K-major)", N, N, T, True, True, f32, 1.0, True),
        ("R2 += Ypre^T A (A K-major)", D, N, T, False, True, f32, 1.0, False),
        ("R1 += Z^T X (row-major copy of Z)", N, D, T, False, False, f32, 1.0, False),
        # other operand layouts: row-major A (fp32-storage path, or when the objective is reported), and transposed
        # copies of Ypre / X that the module does not keep
        ("G_A with A row-major", N, N, T, False, False, f32, 1.0, True),
        ("R2 with A row-major", D, N, T, False, False, f32, 1.0, False),
        ("R2 with Ypre stored transposed too", D, N, T, True, True, f32, 1.0, False),
        ("R1 with X stored transposed", N, D, T, False, True, f32, 1.0, False),
    ]
    for name, M, Nn, K, ak, bk, cdt, beta, lower in cases:
        A = _rnd((M, K) if ak else (K, M), bf)
        # the Gram products multiply a matrix by (the first rows of) itself
        B = A[:Nn] if name.startswith("G_A") and ak and bk else _rnd((Nn, K) if bk else (K, Nn), bf)
        C = _rnd((M, Nn), cdt)
        ms = _timeit(lambda: api.sp_gemm(A, B, C, transA=not ak, transB=bk, alpha=1.0, beta=beta, lower_only=lower,
                                         use_tensor_cores=True, status=st), reps, warm)
        fl = K * Nn * (2.0 * M - Nn) if lower else 2.0 * M * Nn * K     # lower: triangle of the square + rows below it
        print(f"{name:34s} {M:6d} x {Nn:6d} x {K:6d}  {ms:8.3f} ms  {fl / ms / 1e9:8.1f} TFLOP/s", flush=True)
    print("status", st.cpu().tolist())


SOLVE_SIZES = [(2048, 8192), (2048, 4096), (8192, 2048), (4096, 2048)]


def solve_cases(reps, warm):
    st = api.new_status()
    for m, n in SOLVE_SIZES:
        A = torch.relu(torch.randn(n, n + 1024, device=DEV))
        G = (A @ A.T).contiguous()
        del A
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


def mha_case(reps, warm):
    """One sp_mha_step (2 gradient steps of Eq. 85, the closed form of Eq. 86, 2 gradient steps of Eq. 87) on an
    attention module of workload C2's width: d = 2048, 32 heads of 64, 16 sequences of 1024 tokens, 8 per chunk."""
    d, H, T, n_seq, chunk = 2048, 32, 1024, 16, 8
    X = _rnd((n_seq * T, d), torch.bfloat16)
    W = [(torch.randn(d, d, device=DEV) * (1.0 / d ** 0.5)) for _ in range(4)]
    mod = api.MhaModule(X, *W, n_heads=H, T=T, seq_chunk=chunk)
    mod.sp_mha_init(True)
    p = api.MhaParams(a_steps=2, z_steps=2, seq_chunk=chunk)
    ms = _timeit(lambda: mod.sp_mha_step(p), reps, warm)
    api.sp_profile_begin(2)
    mod.sp_mha_step(p)
    torch.cuda.synchronize()
    pr = api.sp_profile_read()
    api.sp_profile_begin(0)
    mod.check_status()
    pairs = n_seq * H
    # batched products per step: logits (1 + z_steps), P V / R V^T (2 a_steps + 1), gradients (2 z_steps), 3 segments
    # where an operand is split; counted once each: 2 T^2 d_h flop per pair
    n_b = (1 + p.z_steps) + (2 * p.a_steps + 1) + 2 * p.z_steps
    fl = n_b * 2.0 * T * T * (d // H) * pairs + 5 * 2.0 * n_seq * T * d * d
    print(f"mha step d={d} H={H} T={T} n_seq={n_seq}: {ms:8.3f} ms  {fl / ms / 1e9:7.1f} TFLOP/s (algorithmic)")
    print("   " + "; ".join(f"{k}: {v['records']} x {1e3 * v['ms'] / max(v['records'], 1):.1f} us"
                            for k, v in pr.items() if v["records"]), flush=True)
    # recovery of W_V: per head the regressors P_i X (2 parts of P), their Gram matrix (3 part products, lower
    # triangle) and the cross product with Aattn_i (3 part products), then one system of size d per head
    ms_v = _timeit(lambda: mod.sp_mha_value_refit(None, 0.05, True), reps, warm)
    api.sp_profile_begin(2)
    mod.sp_mha_value_refit(None, 0.05, True)
    torch.cuda.synchronize()
    pr = api.sp_profile_read()
    api.sp_profile_begin(0)
    mod.check_status()
    fl_v = pairs * (2.0 * T * T * d + 1.0 * d * d * T + 2.0 * (d // H) * d * T) + H * (d ** 3 / 3 + 2.0 * (d // H) * d * d)
    print(f"W_V recovery d={d} H={H} T={T} n_seq={n_seq}: {ms_v:8.3f} ms  {fl_v / ms_v / 1e9:7.1f} TFLOP/s (algorithmic)")
    print("   " + "; ".join(f"{k}: {v['records']} x {1e3 * v['ms'] / max(v['records'], 1):.1f} us"
                            for k, v in pr.items() if v["records"]), flush=True)
    print("status", mod.status.cpu().tolist())


def _timeit_cold(fn, reps, warm, flush):
    """Mean device time of fn() in ms with the L2 overwritten before every call.  The flush (a 1 GiB fill) also keeps
    the stream busy long enough for the host to have queued fn() and the closing event before the GPU gets there."""
    tot = 0.0
    for it in range(warm + reps):
        flush.fill_(it)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        if it >= warm:
            tot += e0.elapsed_time(e1)
    return tot / reps


def mask_cases(reps, warm, hbm_gbs):
    flush = torch.empty(1 << 30, dtype=torch.uint8, device=DEV)

    def line(name, ms, nbytes):
        gbs = nbytes / ms / 1e6
        print(f"{name:58s} {1e3 * ms:9.1f} us  {nbytes / 1e6:9.2f} MB  {gbs:8.1f} GB/s  {gbs / hbm_gbs:5.2f} of HBM peak",
              flush=True)

    # Wanda scores: one pass over the fp32 weight matrix [d, n] (C2, C3 and C5 shapes), channel and head units
    for d, n, group in ((2048, 8192, 1), (4096, 16384, 1), (7168, 28672, 1), (4096, 4096, 128)):
        W = torch.randn(d, n, device=DEV)
        colsq = torch.rand(n, device=DEV)
        colabs = torch.rand(n, device=DEV, dtype=torch.float64)
        nu = n // group
        ws = torch.empty(api.workspace_bytes(api.SP_WS_SCORES, n, 0, d, 0, api.SP_F32), dtype=torch.uint8, device=DEV)
        for kind, nm in ((api.SP_SCORE_WANDA_L2, "L2"), (api.SP_SCORE_WANDA_L1, "L1")):
            ms = _timeit_cold(lambda: api.sp_struct_scores(kind, nu, group, W=W, colsq=colsq, colabs=colabs,
                                                           inv_tokens=1e-5, ws=ws), reps, warm, flush)
            line(f"scores Wanda-{nm}  W [{d}, {n}] fp32, units of {group}", ms, 4.0 * d * n)
        del W
    # Lemma-1 scores streamed from four [N, n] tensors
    for N, n, dt, sz in ((32768, 8192, torch.bfloat16, 2), (16384, 8192, torch.float32, 4)):
        b, c, dd, t = (_rnd((N, n), dt) for _ in range(4))
        ws = torch.empty(api.workspace_bytes(api.SP_WS_SCORES, n, 0, N, 0, api.SP_F32), dtype=torch.uint8, device=DEV)
        ms = _timeit_cold(lambda: api.sp_struct_scores(api.SP_SCORE_LEMMA1, n, 1, b=b, c=c, dd=dd, t=t, ws=ws), reps,
                          warm, flush)
        line(f"scores Lemma-1 streamed  4 x [{N}, {n}] {str(dt)[6:]}", ms, 4.0 * N * n * sz)
        del b, c, dd, t
    # weight statistics of the "-distribute" importances: head slices (rows of W_Q, columns of W_O) and whole MLP matrices
    for rows, cols, axis, group, dt, sz in ((4096, 4096, 0, 128, torch.bfloat16, 2), (4096, 4096, 1, 128, torch.bfloat16, 2),
                                            (16384, 4096, 0, 0, torch.bfloat16, 2), (28672, 7168, 0, 0, torch.bfloat16, 2),
                                            (16384, 4096, 0, 0, torch.float32, 4)):
        W = _rnd((rows, cols), dt)
        nb = 1 if group == 0 else (rows // group if axis == 0 else cols // group)
        st = torch.zeros(nb, 4, dtype=torch.float64, device=DEV)
        ms = _timeit_cold(lambda: api.sp_weight_stats(W, axis, group, st, accumulate=True), reps, warm, flush)
        line(f"weight stats  W [{rows}, {cols}] {str(dt)[6:]}, axis {axis}, blocks of {group}", ms, float(sz) * rows * cols)
        del W
    # allocation over the layers of a model
    for L in (24, 32, 64):
        I = torch.rand(L, dtype=torch.float64, device=DEV) + 0.5
        nu = torch.full((L,), 8192, dtype=torch.int64, device=DEV)
        ms = _timeit_cold(lambda: api.sp_allocate_sparsity(I, nu, 0.5, 1.0), reps, warm, flush)
        line(f"allocate  L = {L}", ms, 32.0 * L)
    # top-k: one layer, and all layers of a model in one launch (4 B score read + 1 B mask written per unit)
    for n, k in ((8192, 4096), (28672, 5734)):
        sc = torch.randn(n, device=DEV)
        ms = _timeit_cold(lambda: api.sp_apply_mask(sc, k, want_index=True), reps, warm, flush)
        line(f"top-k  n = {n}, k = {k}", ms, 9.0 * n)
    for L, n in ((24, 8192), (32, 16384), (32, 28672), (148, 28672)):
        sc = torch.randn(L, n, device=DEV)
        kk = torch.full((L,), n // 2, dtype=torch.int64, device=DEV)
        ms = _timeit_cold(lambda: api.sp_apply_mask_batched(sc, kk), reps, warm, flush)
        line(f"top-k batched  L = {L}, n = {n}", ms, 5.0 * L * n)
    # one threshold over all layers (Algorithm 3): the many-CTA select, and the one-CTA select over the same keys
    for L, n in ((4, 8192), (24, 8192), (32, 16384), (32, 28672)):
        sc = torch.randn(L, n, device=DEV)
        msk = torch.empty(L, n, dtype=torch.uint8, device=DEV)
        ms = _timeit_cold(lambda: api.sp_apply_mask_global(sc, 0.4, 1, mask_out=msk), reps, warm, flush)
        line(f"global threshold, many CTAs  L = {L}, n = {n}", ms, 25.0 * L * n)
        K = int(0.4 * n * L)
        ms = _timeit_cold(lambda: api.sp_apply_mask(sc.view(-1), K, mask_out=msk.view(-1)), reps, warm, flush)
        line(f"global threshold, one CTA    L = {L}, n = {n}", ms, 25.0 * L * n)


def lockstep_cases(reps, warm, layers=4, tokens=32768):
    """Iterations of the lock-step run (all layers' scores, one global threshold, all layers' fixed-mask steps) on
    `layers` modules of C2's width with `tokens` tokens each, against the same modules stepped one by one with
    per-layer top-k (the ordinary step)."""
    from . import pipeline, synth
    cfg = synth.scaled(synth.CONFIGS["C2"], tokens=tokens, layers=layers)
    data = []
    for l in range(layers):
        X = synth.make_activations(cfg, l).to(DEV)
        W1, W2 = (w.to(DEV) * (1.0 + 0.03 * l) for w in synth.make_weights(cfg, l))
        data.append((X, W1, W2))
    keep = 1.0 - cfg.sparsity
    results, scores, masks = pipeline.prune_ffn_layers_global(lambda l: data[l], layers, cfg.n, keep, 2,
                                                              params=api.AdmmParams(rho=cfg.rho), token_chunk=32768)
    torch.cuda.synchronize()
    counts = masks.sum(dim=1).cpu().tolist()
    K = int(keep * cfg.n * layers + 1e-9)
    del results
    print(f"lock-step: {layers} layers x {tokens} tokens, d={cfg.d}, n={cfg.n}, kept fraction {keep}: kept per layer "
          f"after 2 iterations {counts}")
    sel = _timeit(lambda: api.sp_apply_mask(scores.view(-1), K, mask_out=masks.view(-1)), max(reps, 10), warm)
    print(f"global select over {layers * cfg.n} scores (K = {K}): {sel * 1e3:.0f} us")
    # the ordinary step on the same modules, per-layer top-k with the lock-step run's final counts
    mods = []
    for l in range(layers):
        m = api.FfnModule(*data[l], token_chunk=32768, overlap_k=int(counts[l]))
        m.sp_ffn_init()
        mods.append(m)

    def ordinary():
        for l, m in enumerate(mods):
            m.sp_admm_step(api.AdmmParams(rho=cfg.rho, k_keep=int(counts[l]), token_chunk=32768))
    ms = _timeit(ordinary, reps, warm)
    print(f"ordinary steps (per-layer top-k, same kept counts): {ms:.2f} ms per iteration of all layers")

    def lock():
        pl = api.AdmmParams(rho=cfg.rho, k_keep=1, token_chunk=32768)
        for m in mods:
            m.sp_admm_scores(pl)
        for l, m in enumerate(mods):
            m.sp_admm_step(api.AdmmParams(rho=cfg.rho, k_keep=int(counts[l]), token_chunk=32768, reselect_mask=False,
                                          skip_scores=True))
    ms2 = _timeit(lock, reps, warm)
    print(f"lock-step calls on the same modules (scores of all layers, then fixed-mask steps; select not included): "
          f"{ms2:.2f} ms per iteration of all layers")


def _hbm_peak():
    import json
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["gemm", "solve", "mask", "lockstep", "mha"])
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--warm", type=int, default=2)
    ap.add_argument("--sizes", default="", help="solve: m:n pairs, e.g. 7168:28672,4096:16384 (default: those of a C2 step)")
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("microbench needs a CUDA device")
    api.lib()
    if a.what == "mask":
        peak, src = _hbm_peak()
        print(f"HBM peak {peak:.0f} GB/s ({src})")
        mask_cases(a.reps, a.warm, peak)
    elif a.what == "lockstep":
        lockstep_cases(a.reps, a.warm)
    else:
        if a.what == "mha":
            mha_case(a.reps, a.warm)
            return
        if a.sizes:
            SOLVE_SIZES[:] = [tuple(int(v) for v in pair.split(":")) for pair in a.sizes.split(",")]
        (gemm_cases if a.what == "gemm" else solve_cases)(a.reps, a.warm)


if __name__ == "__main__":
    main()
