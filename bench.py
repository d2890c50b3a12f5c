#!/usr/bin/env python
"""Benchmark of the per-module ADMM path (STRUPRUNE hot path) on B200.

A step = one pass of the whole hot path over one FFN module: sp_admm_step (weight recovery by Cholesky solves, unit
scores, top-k mask, recovery on the kept support, a-/z-(dual-)updates and Gram / cross-product accumulation over all
calibration tokens) followed by sp_allocate_sparsity over the model's layer importances.

Workload at N = 1 GPU: workload C2 (OPT-1.3B-shaped FFN module: d = 2048, n = 8192, 128 x 2048 = 262144
calibration tokens in bf16, 50 % channel sparsity), synthetic seeded inputs generated on the device.
With N > 1 GPUs every rank owns its own module (modules are independent once the kept counts are fixed), so the
scaling is weak and the data path has no collective.  `--shard tokens` instead splits the tokens of ONE module over
the ranks (strong scaling; the accumulators are all-reduced once per iteration).

Prints ONE JSON line (rank 0).  Besides the timed step (mask re-selected in every iteration) the line carries
`fixed_mask` (the same module stepped without re-selection, and its continuation on the kept channels only), `e2e`
(one whole pruned layer from and to pinned host buffers: the FFN module's iterations and the attention half with fixed
head outputs) and `cpu_baseline` (the oracle on a token sample).  `--dual` runs with the scaled dual variable.
`--impl reference` times the CPU oracle instead (a deliberately plain fp64 restatement of the paper; context only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ADMM iterations/sec per module"
UNIT = "iterations/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C2")
    ap.add_argument("--tokens", type=int, default=0, help="override the token count (profiling on a small case)")
    ap.add_argument("--chunk", type=int, default=32768)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fixed-mask", action="store_true", help="skip the fixed-mask variants of the step")
    ap.add_argument("--dual", action="store_true", help="run with the scaled dual variable U (dual_mode = 1)")
    ap.add_argument("--shard", default="modules", choices=["modules", "tokens"],
                    help="N > 1: every rank its own module (default, no collective), or ONE module with its tokens "
                         "split over the ranks (accumulators all-reduced once per iteration)")
    ap.add_argument("--cpu-sample-tokens", type=int, default=1024)
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------ reference arm
def oracle_iteration_seconds(cfg, sample_tokens: int, repeats: int = 1):
    """Times one oracle ADMM iteration at the config's d and n on `sample_tokens` tokens.  Returns the seconds of the
    token-independent weight phase and of the token-dependent phase (a-, z-update, accumulators)."""
    import numpy as np
    from oracle import struprune_oracle as O
    from paper_2510_03246_b200 import synth

    X = synth.make_activations(cfg, tokens=sample_tokens).double().numpy().T.copy()
    W1, W2 = synth.make_weights(cfg)
    W1 = W1.double().numpy(); W2 = W2.double().numpy()
    gated = cfg.act == "swiglu"
    if gated:
        st, Y = O.swiglu_init(X, synth.make_gate_weights(cfg).double().numpy(), W1, W2)
    else:
        st, Y = O.ffn_init(X, W1, W2)
    p = O.AdmmParams(k_keep=cfg.k_keep, rho=cfg.rho, act=cfg.act)
    tw = tt = 0.0
    for _ in range(repeats):
        t0 = time.perf_counter()
        O.admm_weight_phase(st, W1, p, X.shape[1])
        t1 = time.perf_counter()
        A = O.a_update(st.W2, Y, st.Z, p.alpha, p.beta, None, cfg.act, st.gate)
        z1, z2 = O.z_candidates(st.W1, X, A, p.alpha, p.beta)
        st.Z = (O.swiglu_zu_update(A, st.gate, z1, p.alpha, p.beta) if gated
                else O.z_select(st.Z, z1, z2, A, p.alpha, p.beta, p.z_rule))
        st.G_A = A @ A.T; st.R1 = st.Z @ X.T; st.R2 = Y @ A.T; st.absA = np.abs(A).sum(axis=1)
        O.allocate_sparsity(np.linspace(1.0, 1.5, cfg.layers), [cfg.n] * cfg.layers, cfg.sparsity, 1.25)
        t2 = time.perf_counter()
        tw += t1 - t0
        tt += t2 - t1
    return tw / repeats, tt / repeats


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 0) for d in threadpool_info()]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def cpu_baseline(cfg, sample_tokens: int) -> dict:
    tw, tt = oracle_iteration_seconds(cfg, sample_tokens)
    full = tw + tt * (cfg.tokens / sample_tokens)
    return {"value": 1.0 / full, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
            "sample": (f"one oracle iteration at d={cfg.d}, n={cfg.n} on {sample_tokens} of {cfg.tokens} tokens "
                       f"({tw + tt:.1f} s measured: weight phase {tw:.1f} s + token phase {tt:.1f} s); the token "
                       f"phase is scaled x{cfg.tokens // sample_tokens} to the full token count (extrapolated)")}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    for _ in range(min(args.warmup, 1)):
        oracle_iteration_seconds(cfg, args.cpu_sample_tokens)
    t0 = time.perf_counter()
    tws = tts = 0.0
    steps = max(1, args.steps)
    for _ in range(steps):
        tw, tt = oracle_iteration_seconds(cfg, args.cpu_sample_tokens)
        tws += tw; tts += tt
    tw, tt = tws / steps, tts / steps
    full = tw + tt * (cfg.tokens / args.cpu_sample_tokens)
    value = 1.0 / full
    sample = (f"each step: one oracle iteration at d={cfg.d}, n={cfg.n} on {args.cpu_sample_tokens} of {cfg.tokens} "
              f"tokens; token phase scaled x{cfg.tokens // args.cpu_sample_tokens} (extrapolated)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": 1e3 * full, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfg)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": time.perf_counter() - t0}
    print(json.dumps(line))


def workload_name(cfg) -> str:
    shape = {"C1": "OPT-125M", "C2": "OPT-1.3B", "C3": "OPT-6.7B", "C4": "LLaMA-2-7B", "C5": "OPT-30B"}.get(cfg.name, "OPT")
    kind = "SwiGLU FFN module (gate/up/down)" if cfg.act == "swiglu" else "FFN module"
    return (f"{cfg.name}: {shape}-shaped {kind}, d={cfg.d}, n={cfg.n}, N={cfg.tokens} tokens, "
            f"{cfg.storage} activations, {int(cfg.sparsity * 100)}% channel sparsity (k_keep={cfg.k_keep})")


# ------------------------------------------------------------------------------------------------ our arm
def main():
    args = parse()
    from paper_2510_03246_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.tokens:
        cfg = synth.scaled(cfg, tokens=args.tokens)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2510_03246_b200 import api, parallel

    rank, local_rank, world = parallel.env_world()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    api.lib()

    # ---- inputs resident in HBM: this rank's module (layer index = rank), or its token shard of module 0
    by_tokens = args.shard == "tokens"
    if by_tokens and cfg.act == "swiglu":
        raise SystemExit("--shard tokens: ReLU modules only")
    layer = rank
    wl = 0 if by_tokens else layer
    cfg_local = synth.scaled(cfg, tokens=cfg.tokens // world) if by_tokens else cfg
    X = synth.make_activations(cfg_local, layer, device=dev)        # another seed per rank: disjoint tokens
    W1_0, W2_0 = synth.make_weights(cfg, wl, device=dev)
    Wg_0 = synth.make_gate_weights(cfg, layer, device=dev) if cfg.act == "swiglu" else None
    mod = api.FfnModule(X, W1_0, W2_0, dual_mode=args.dual, token_chunk=args.chunk, overlap_k=cfg.k_keep, Wg_0=Wg_0)
    I_all = synth.make_importances(cfg, device=dev)
    n_units = torch.full((cfg.layers,), cfg.n, dtype=torch.int64, device=dev)
    T_soft = float(I_all.abs().mean())
    if by_tokens:
        parallel.token_sharded_init([mod])
    else:
        mod.sp_ffn_init()
    torch.cuda.synchronize()
    mod.check_status()
    prm = api.AdmmParams(k_keep=cfg.k_keep, rho=cfg.rho, token_chunk=args.chunk, dual_mode=args.dual)

    def step():
        if by_tokens:
            parallel.token_sharded_iterations([mod], prm, 1, read_reports=False)
        else:
            mod.sp_admm_step(prm)
        # layer importances -> per-layer kept counts (this module's own importance replaces its slot)
        I_all[layer:layer + 1].copy_(mod.importance)
        api.sp_allocate_sparsity(I_all, n_units, cfg.sparsity, T_soft)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    mod.check_status()

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    api.sp_profile_begin(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ms_local = ev0.elapsed_time(ev1)
    launches = api.sp_launch_count()
    prof = api.sp_profile_read()
    api.sp_profile_begin(False)
    mod.check_status()
    ms = parallel.max_over_ranks(ms_local, dev)
    value = (1 if by_tokens else world) * args.steps / (ms * 1e-3)      # one module in all when its tokens are split

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the tcgen05 GEMM), from CUDA events recorded around each launch
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    # launches that own the whole GPU, and the z1 products that run on a subset of the SM pairs beside the recovery
    # on the kept support (their durations are stretched by design); the roofline figure covers both
    tc_own, tc_sh = prof["gemm_tc"], prof.get("gemm_tc_shared", {"records": 0, "ms": 0.0, "flops": 0.0, "bytes": 0.0})
    tc = {k: tc_own[k] + tc_sh[k] for k in ("records", "ms", "flops")}
    peak_tf = peaks.get("bf16_tflops_sustained", 1400.0)
    peak_src = "measured (sustained, MEASURED_PEAKS.json)" if peaks else "fallback (1.4 PFLOP/s sustained)"
    achieved = tc["flops"] / (tc["ms"] * 1e-3) / 1e12 if tc["ms"] > 0 else 0.0
    # DRAM traffic of the token-pass GEMMs from the ncu capture in profiles/gemm_tc_kernel_C2_one_chunk.md: the six
    # products of one 16384-token chunk of C2 moved 4.22 GB; traffic grows in proportion to the tokens a launch covers.
    traffic = None
    if cfg.name == "C2" and cfg.d == 2048 and cfg.n == 8192 and cfg.k_keep == 4096 and tc["records"]:
        traffic = 4.22e9 * (cfg.tokens / 16384.0) * args.steps / tc["records"]
    roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel", "achieved": achieved, "peak": peak_tf,
                "unit": "TFLOP/s", "frac": achieved / peak_tf, "traffic": traffic,
                "traffic_unit": "DRAM bytes per launch (ncu, one chunk, scaled by tokens)", "peak_source": peak_src,
                "launches": tc["records"], "avg_launch_ms": tc["ms"] / max(tc["records"], 1),
                "algorithmic_flops_per_launch": tc["flops"] / max(tc["records"], 1),
                "launches_owning_gpu": tc_own["records"],
                "achieved_owning_gpu": tc_own["flops"] / (tc_own["ms"] * 1e-3) / 1e12 if tc_own["ms"] > 0 else 0.0}
    hbm = peaks.get("hbm_gbs", 6650.0)
    fu = prof["fused_update"]
    # DRAM traffic of one fused-update launch from the ncu capture in profiles/fused_update_prep_h_C2_one_chunk.md:
    # 2.148 GB read + 2.124 GB written for one 32768-token chunk of C2 without the dual variable (algorithmic 4.29 GB)
    fu_traffic = None
    if (cfg.name == "C2" and cfg.n == 8192 and cfg.k_keep == 4096 and args.chunk == 32768 and not args.dual
            and cfg.tokens % args.chunk == 0):
        fu_traffic = 4.272e9
    roofline_hbm = {"bound": "hbm", "kernel": "fused_update_kernel",
                    "achieved": fu["bytes"] / (fu["ms"] * 1e-3) / 1e9 if fu["ms"] else 0.0, "peak": hbm, "unit": "GB/s",
                    "frac": (fu["bytes"] / (fu["ms"] * 1e-3) / 1e9 / hbm) if fu["ms"] else 0.0, "traffic": fu_traffic,
                    "algorithmic_bytes_per_launch": fu["bytes"] / max(fu["records"], 1),
                    "launches": fu["records"]}
    breakdown = {k: {"records": v["records"], "ms_per_step": v["ms"] / args.steps,
                     **({"tflops": v["flops"] / (v["ms"] * 1e-3) / 1e12} if v["flops"] and v["ms"] else {}),
                     **({"gbs": v["bytes"] / (v["ms"] * 1e-3) / 1e9, "hbm_frac": v["bytes"] / (v["ms"] * 1e-3) / 1e9 / hbm}
                        if v["bytes"] and v["ms"] else {})}
                 for k, v in prof.items() if v["records"]}

    # ---- the variant with the mask fixed after the first iterations (Algorithm 1: Step 3 fixes the masks before the
    # SparseLLM iterations): the same module stepped without re-selection, and its continuation on the kept channels
    fixed = None
    if not args.no_fixed_mask and rank == 0:
        from paper_2510_03246_b200 import pipeline

        def time_steps(m, prm_v, n_warm=2, n_timed=4):
            for _ in range(n_warm):
                m.sp_admm_step(prm_v)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for _ in range(n_timed):
                m.sp_admm_step(prm_v)
            b.record()
            torch.cuda.synchronize()
            m.check_status()
            return a.elapsed_time(b) / n_timed

        api.sp_profile_begin(0)
        prm_fix = api.AdmmParams(k_keep=cfg.k_keep, rho=cfg.rho, token_chunk=args.chunk, reselect_mask=False,
                                 skip_scores=True, dual_mode=args.dual)
        ms_full = time_steps(mod, prm_fix)
        cmod, _ = pipeline.compact_module(mod)
        ms_comp = time_steps(cmod, prm_fix)
        del cmod
        torch.cuda.empty_cache()
        fixed = {"note": "steps with the mask kept fixed (no unrestricted recovery, no scores): on the full-width "
                         "module, and continued on the kept channels only (accumulators k x k)",
                 "full_width_ms_per_step": ms_full, "full_width_iterations_per_s": 1e3 / ms_full,
                 "kept_channels_ms_per_step": ms_comp, "kept_channels_iterations_per_s": 1e3 / ms_comp}

    # ---- end to end: host buffers in, host results out, one whole module job of cfg.iters iterations
    e2e = None
    if not args.no_e2e:
        del mod
        torch.cuda.empty_cache()
        hX = X.cpu().pin_memory(); hW1 = W1_0.cpu().pin_memory(); hW2 = W2_0.cpu().pin_memory()
        hWg = Wg_0.cpu().pin_memory() if Wg_0 is not None else None
        del X, W1_0, W2_0, Wg_0
        torch.cuda.empty_cache()
        iters = cfg.iters
        # the attention half of the layer: fixed head outputs H and the output projection W_O (host, pinned)
        from paper_2510_03246_b200 import pipeline
        hH, hWo = synth.make_attention_inputs(cfg, layer)
        hH = hH.pin_memory(); hWo = hWo.pin_memory()
        k_heads = max(1, cfg.heads - int(cfg.heads * cfg.sparsity + 0.5))
        # results come back into pinned host buffers
        oW1 = torch.empty(cfg.n, cfg.d, dtype=torch.float32).pin_memory(); oW2 = torch.empty(cfg.d, cfg.n, dtype=torch.float32).pin_memory()
        omask = torch.empty(cfg.n, dtype=torch.uint8).pin_memory()
        oWo = torch.empty(cfg.d, cfg.d, dtype=torch.float32).pin_memory(); ohm = torch.empty(cfg.heads, dtype=torch.uint8).pin_memory()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        dX = hX.to(dev, non_blocking=True); dW1 = hW1.to(dev, non_blocking=True); dW2 = hW2.to(dev, non_blocking=True)
        dWg = hWg.to(dev, non_blocking=True) if hWg is not None else None
        m2 = api.FfnModule(dX, dW1, dW2, dual_mode=args.dual, token_chunk=args.chunk, overlap_k=cfg.k_keep, Wg_0=dWg)
        m2.sp_ffn_init()
        # this layer's share of pass 0: the importance of the pre-trained module
        api.sp_struct_scores(api.SP_SCORE_WANDA_L2, cfg.n, W=m2.W2_0, colsq=m2.G_A, colsq_stride=cfg.n + 1)
        for _ in range(iters):
            m2.sp_admm_step(prm)
        oW1.copy_(m2.W1, non_blocking=True); oW2.copy_(m2.W2, non_blocking=True); omask.copy_(m2.mask, non_blocking=True)
        torch.cuda.synchronize()
        t_ffn = time.perf_counter()
        # attention module: pre-trained output of the projection, head scores, head mask, W_O recovery on the kept heads
        dH = hH.to(dev, non_blocking=True); dWo = hWo.to(dev, non_blocking=True)
        Ya = torch.empty(dH.shape[0], cfg.d, dtype=dH.dtype, device=dev)
        api.sp_gemm(dH, dWo, Ya, transB=True, use_tensor_cores=(dH.dtype == torch.bfloat16))
        hmask, Wo_new, _ = pipeline.prune_attention_heads(dH, Ya, dWo.float(), cfg.heads, k_heads, rho=cfg.rho,
                                                          token_chunk=args.chunk)
        oWo.copy_(Wo_new, non_blocking=True); ohm.copy_(hmask, non_blocking=True)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        m2.check_status()
        h2d = hX.numel() * hX.element_size() + hW1.numel() * hW1.element_size() + hW2.numel() * hW2.element_size()
        if hWg is not None:
            h2d += hWg.numel() * hWg.element_size()
        h2d += hH.numel() * hH.element_size() + hWo.numel() * hWo.element_size()
        d2h = oW1.numel() * 4 + oW2.numel() * 4 + omask.numel() + oWo.numel() * 4 + ohm.numel()
        e2e = {"value": iters / (t1 - t0), "unit": UNIT, "layers_per_s": 1.0 / (t1 - t0), "h2d_bytes_per_step": h2d / iters,
               "d2h_bytes_per_step": d2h / iters, "iterations": iters, "ffn_seconds": t_ffn - t0,
               "attention_seconds": t1 - t_ffn,
               "note": "one pruned layer: pinned-host X, W1_0, W2_0 in; init + importance of the pre-trained module + "
                       "iterations; W1, W2, mask back to host; then the attention half with fixed head outputs (H, "
                       "W_O in; head scores, head mask, W_O recovery on the kept heads; W_O, mask out); "
                       "layers_per_s is that whole job per second, value = iterations / that time"}

    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, args.cpu_sample_tokens)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong" if by_tokens else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "token_chunk": args.chunk, "dual_mode": bool(args.dual),
                       "l2": "inputs larger than L2 (Z alone is %.1f GB)" % (cfg.tokens * cfg.n * 4 / 1e9),
                       "parallelism": (f"tokens x{world} of one module (accumulators all-reduced once per iteration)"
                                       if by_tokens else f"modules x{world} (independent, no collective)")},
            "clocks": clocks, "gpu_launches": launches, "roofline": roofline, "roofline_hbm": roofline_hbm, "e2e": e2e, "cpu_baseline": cpu, "fixed_mask": fixed,
            "breakdown": breakdown}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
