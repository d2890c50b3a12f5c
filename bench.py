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
head outputs), `attention_module` (the attention module's step under the second MHA objective and the recovery of
W_V, timed on 16 sequences of 1024 tokens at the workload's width) and `cpu_baseline` (the oracle on a token sample).
`--dual` runs with the scaled dual variable.
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
DTYPE_NAME = {"bf16": "bf16", "f32": "f32"}
WORKLOAD_GB = {"C1": 1, "C2": 40, "C3": 60, "C4": 110, "C5": 160}    # free device memory a workload needs


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
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing of the step")
    ap.add_argument("--reproducible", action="store_true",
                    help="run with sp_set_reproducible(1): fixed summation order, bit-identical results")
    ap.add_argument("--cpu-sample-tokens", type=int, default=1024)
    ap.add_argument("--workloads", default="C3,C4,C5",
                    help="1 GPU: further workloads measured after the main one and reported under `workloads` "
                         "(empty string: none)")
    ap.add_argument("--no-pruned-decay", action="store_true",
                    help="do not keep the ordered accumulators that let a step scale, instead of recompute, the parts of "
                         "G_A and R2 that belong to pruned channels while the mask stays")
    ap.add_argument("--no-attention", action="store_true",
                    help="skip the timing of the attention module's step and W_V recovery (`attention_module`)")
    ap.add_argument("--workload-steps", type=int, default=5)
    ap.add_argument("--workload-warmup", type=int, default=2)
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
            "implementation": "numpy fp64 (LAPACK / BLAS on all threads counted in cores)",
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
            "config": config_dict(cfg, args, int(os.environ.get("WORLD_SIZE", 1)), args.shard == "tokens"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                             "implementation": "numpy fp64 (LAPACK / BLAS on all threads counted in cores)",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": time.perf_counter() - t0}
    print(json.dumps(line))


def config_dict(cfg, args, world: int, by_tokens: bool) -> dict:
    """The `config` object of the JSON line; both arms describe the workload with the same one."""
    return {"workload": workload_name(cfg), "token_chunk": args.chunk, "dual_mode": bool(args.dual),
            "reproducible": bool(args.reproducible),
            "l2": "inputs larger than L2 (Z alone is %.1f GB)" % (cfg.tokens * cfg.n * 4 / 1e9),
            "parallelism": (f"tokens x{world} of one module (accumulators all-reduced once per iteration)"
                            if by_tokens else f"modules x{world} (independent, no collective)")}


def workload_name(cfg) -> str:
    shape = {"C1": "OPT-125M", "C2": "OPT-1.3B", "C3": "OPT-6.7B", "C4": "LLaMA-2-7B", "C5": "OPT-30B"}.get(cfg.name, "OPT")
    kind = "SwiGLU FFN module (gate/up/down)" if cfg.act == "swiglu" else "FFN module"
    return (f"{cfg.name}: {shape}-shaped {kind}, d={cfg.d}, n={cfg.n}, N={cfg.tokens} tokens, "
            f"{cfg.storage} activations, {int(cfg.sparsity * 100)}% channel sparsity (k_keep={cfg.k_keep})")


# ------------------------------------------------------------------------------------------------ our arm
def load_peaks():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        return {}


def captured_traffic(kernel: str, key: str):
    """DRAM bytes of one launch group from the ncu captures summarised under profiles/ (profiles/ncu_dram_traffic.txt:
    JSON, one record per captured kernel with the sha256 of the source file it was built from).  Returns None when no
    record matches or when the kernel's source has changed since the capture (the counters are then stale)."""
    import hashlib
    try:
        recs = json.load(open(os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")))["records"]
    except Exception:
        return None
    for r in recs:
        if r.get("kernel") == kernel and r.get("key") == key:
            try:
                src = open(os.path.join(ROOT, r["source"]), "rb").read()
            except Exception:
                return None
            return r["dram_bytes"] if hashlib.sha256(src).hexdigest() == r.get("source_sha256") else None
    return None


def build_module(cfg, args, dev, layer, by_tokens, world):
    import torch
    from paper_2510_03246_b200 import api, parallel, synth
    wl = 0 if by_tokens else layer
    cfg_local = synth.scaled(cfg, tokens=cfg.tokens // world) if by_tokens else cfg
    X = synth.make_activations(cfg_local, layer, device=dev)        # another seed per rank: disjoint tokens
    W1_0, W2_0 = synth.make_weights(cfg, wl, device=dev)
    Wg_0 = synth.make_gate_weights(cfg, layer, device=dev) if cfg.act == "swiglu" else None
    mod = api.FfnModule(X, W1_0, W2_0, dual_mode=args.dual, token_chunk=args.chunk, overlap_k=cfg.k_keep, Wg_0=Wg_0,
                        pruned_decay=not args.no_pruned_decay)
    if by_tokens:
        parallel.token_sharded_init([mod])
    else:
        mod.sp_ffn_init()
    torch.cuda.synchronize()
    mod.check_status()
    return mod, X, W1_0, W2_0, Wg_0


def measure(cfg, args, dev, mod, layer, by_tokens, world, steps, warmup, local_rank, graph=False):
    """Times `steps` steps of the module (profiling off: nothing but the library's own launches in the timed region),
    then the same number of steps again with a CUDA event pair around every launch / phase for the per-kernel figures.
    Returns (ms of the timed loop on this rank, launches in it, clocks, per-kind event records, ms of the profiled loop)."""
    import torch
    import torch.distributed as dist
    from paper_2510_03246_b200 import api, parallel, synth
    I_all = synth.make_importances(cfg, device=dev)
    n_units = torch.full((cfg.layers,), cfg.n, dtype=torch.int64, device=dev)
    T_soft = float(I_all.abs().mean())
    prm = api.AdmmParams(k_keep=cfg.k_keep, rho=cfg.rho, token_chunk=args.chunk, dual_mode=args.dual)
    slot = layer % cfg.layers

    def step():
        if by_tokens:
            parallel.token_sharded_iterations([mod], prm, 1, read_reports=False)
        else:
            mod.sp_admm_step(prm)
        # layer importances -> per-layer kept counts (this module's own importance replaces its slot)
        I_all[slot:slot + 1].copy_(mod.importance)
        api.sp_allocate_sparsity(I_all, n_units, cfg.sparsity, T_soft)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    mod.check_status()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    api.sp_profile_begin(0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ms_local = ev0.elapsed_time(ev1)
    launches = api.sp_launch_count()
    mod.check_status()
    # the same steps replayed from a CUDA graph (one captured step; the library's forks onto its own streams are
    # event-ordered and capture with it): what a caller gains who captures the loop body
    graph_ms = None
    if graph and not by_tokens:
        try:
            cap = torch.cuda.Stream()
            cap.wait_stream(torch.cuda.current_stream())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap, capture_error_mode="relaxed"):
                step()
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            ev0.record()
            for _ in range(steps):
                g.replay()
            ev1.record()
            torch.cuda.synchronize()
            graph_ms = ev0.elapsed_time(ev1) / steps
            mod.check_status()
            del g
        except Exception as exc:   # capture is optional: report why it was not taken
            graph_ms = f"not captured: {type(exc).__name__}"
    # second loop: the same steps with events around every launch
    api.sp_profile_begin(True)
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    prof = api.sp_profile_read()
    api.sp_profile_begin(False)
    mod.check_status()
    return ms_local, launches, clocks, prof, ev0.elapsed_time(ev1), prm, graph_ms


def rooflines(cfg, args, prof, steps, peaks):
    """Roofline records of the dominant kernel (tcgen05 GEMM, tensor bound) and of the fused update (HBM bound) from the
    per-launch CUDA events, plus the per-kind breakdown."""
    # launches that own the whole GPU, and the z1 products that run on a subset of the SM pairs beside the recovery
    # on the kept support (their durations are stretched by design); the roofline figure covers both
    tc_own, tc_sh = prof["gemm_tc"], prof.get("gemm_tc_shared", {"records": 0, "ms": 0.0, "flops": 0.0, "bytes": 0.0})
    tc = {k: tc_own[k] + tc_sh[k] for k in ("records", "ms", "flops")}
    peak_tf = peaks.get("bf16_tflops_sustained", 1400.0)
    peak_src = "measured (sustained, MEASURED_PEAKS.json)" if peaks else "fallback (1.4 PFLOP/s sustained)"
    achieved = tc["flops"] / (tc["ms"] * 1e-3) / 1e12 if tc["ms"] > 0 else 0.0
    # DRAM traffic of the token-pass GEMMs: captured with ncu on one 16384-token chunk; the traffic of each of these
    # products grows in proportion to the tokens it covers
    traffic = None
    t16 = captured_traffic("gemm_tc_kernel", f"{cfg.name}:d={cfg.d},n={cfg.n},k={cfg.k_keep},tokens=16384")
    if t16 is not None and tc["records"]:
        traffic = t16 * (cfg.tokens / 16384.0) * steps / tc["records"]
    roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel", "achieved": achieved, "peak": peak_tf,
                "unit": "TFLOP/s", "frac": achieved / peak_tf, "traffic": traffic,
                "traffic_unit": "DRAM bytes per launch (ncu, one chunk, scaled by tokens)", "peak_source": peak_src,
                "launches": tc["records"], "avg_launch_ms": tc["ms"] / max(tc["records"], 1),
                "algorithmic_flops_per_launch": tc["flops"] / max(tc["records"], 1),
                "launches_owning_gpu": tc_own["records"],
                "achieved_owning_gpu": tc_own["flops"] / (tc_own["ms"] * 1e-3) / 1e12 if tc_own["ms"] > 0 else 0.0}
    hbm = peaks.get("hbm_gbs", 6650.0)
    fu = prof["fused_update"]
    fu_traffic = None
    # ReLU modules without the dual variable that hold the ordered accumulators run the form of the update that also
    # writes the next step's operands (the transposed bf16 copy of Z and h)
    writes_next = (cfg.storage == "bf16" and cfg.act == "relu" and not args.dual and not args.no_pruned_decay
                   and cfg.n % 4 == 0 and cfg.tokens % 8 == 0 and args.chunk % 8 == 0)
    fu_kernel = "fused_update_next_kernel" if writes_next else "fused_update_kernel"
    if args.chunk == 32768 and not args.dual and cfg.tokens % args.chunk == 0:
        fu_traffic = captured_traffic(fu_kernel, f"{cfg.name}:n={cfg.n},k={cfg.k_keep},tokens=32768")
    fu_gbs = fu["bytes"] / (fu["ms"] * 1e-3) / 1e9 if fu["ms"] else 0.0
    # bytes the two elementwise kernels of the token pass move per token (their own algorithmic counts), against the
    # minimum of a pass that reads X, Ypre, Z once and writes Z once in the storage type: s (2 d + 2 n)
    ph = prof.get("prep_h", {"bytes": 0.0})
    esz = 2.0 if cfg.storage == "bf16" else 4.0
    per_token = (fu["bytes"] + ph["bytes"]) / max(steps, 1) / cfg.tokens
    minimum = esz * (2.0 * cfg.d + 2.0 * cfg.n)
    roofline_hbm = {"bound": "hbm", "kernel": fu_kernel, "achieved": fu_gbs, "peak": hbm, "unit": "GB/s",
                    "frac": fu_gbs / hbm, "traffic": fu_traffic,
                    "algorithmic_bytes_per_launch": fu["bytes"] / max(fu["records"], 1), "launches": fu["records"],
                    "elementwise_bytes_per_token": per_token, "minimum_bytes_per_token": minimum,
                    "bytes_over_minimum": per_token / minimum,
                    "bytes_note": "elementwise_bytes_per_token: h gather (none while the mask stays when the update "
                                  "leaves h for the next step) + fused update (Z kept in fp32, A and a storage copy of "
                                  "Z written for the accumulator products, D and z1 read); minimum: X, Ypre, Z read "
                                  "once and Z written once in the storage type",
                    "peak_source": "measured (MEASURED_PEAKS.json)" if peaks else "fallback (6.65 TB/s)"}
    breakdown = {k: {"records": v["records"], "ms_per_step": v["ms"] / steps,
                     **({"tflops": v["flops"] / (v["ms"] * 1e-3) / 1e12} if v["flops"] and v["ms"] else {}),
                     **({"gbs": v["bytes"] / (v["ms"] * 1e-3) / 1e9, "hbm_frac": v["bytes"] / (v["ms"] * 1e-3) / 1e9 / hbm}
                        if v["bytes"] and v["ms"] else {})}
                 for k, v in prof.items() if v["records"]}
    return roofline, roofline_hbm, breakdown


def attention_module_timing(cfg, dev, n_seq=16, T=1024, seq_chunk=8, steps=3):
    """The attention half of a layer of the workload's width under the paper's second MHA objective: sp_mha_step (two
    gradient steps of Eq. 85, the closed form of Eq. 86, two gradient steps of Eq. 87) and the recovery of W_V
    (sp_mha_value_refit), on n_seq synthetic sequences of T tokens, timed with CUDA events after one warm-up call.
    Not part of `value`: the headline metric counts iterations of the FFN module."""
    import torch
    from paper_2510_03246_b200 import api, synth
    d, H = cfg.d, cfg.heads
    acfg = synth.scaled(cfg, tokens=n_seq * T, outlier_frac=0.0)
    X = synth.make_activations(acfg, 0).to(dev)
    W = []
    for tid in (11, 12, 13, 14):
        w = synth.standard_variates(synth.module_seed(acfg, 0), tid, d * d, "gauss").view(d, d)
        W.append((w * (1.2 / d ** 0.5)).to(dev))
    mod = api.MhaModule(X, *W, n_heads=H, T=T, seq_chunk=seq_chunk)
    mod.sp_mha_init(True)
    prm = api.MhaParams(a_steps=2, z_steps=2, seq_chunk=seq_chunk)

    def timed(fn):
        fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        mod.check_status()
        return a.elapsed_time(b) / steps

    ms_step = timed(lambda: mod.sp_mha_step(prm))
    ms_refit = timed(lambda: mod.sp_mha_value_refit(None, cfg.rho, True))
    out = {"workload": f"attention module d={d}, {H} heads of {d // H}, {n_seq} sequences of {T} tokens "
                       f"({seq_chunk} per chunk), bf16, causal",
           "mha_step_ms": ms_step, "mha_step_note": "2 gradient steps of Eq. (85), Eq. (86) in closed form, 2 gradient "
                                                    "steps of Eq. (87); accumulators of the recoveries rebuilt",
           "value_refit_ms": ms_refit, "value_refit_note": "W_V from P and Aattn: one ridge system of size d per head",
           "tokens": n_seq * T}
    del mod, X, W
    torch.cuda.empty_cache()
    return out


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
    if args.reproducible:
        api.sp_set_reproducible(True)

    # ---- inputs resident in HBM: this rank's module (layer index = rank), or its token shard of module 0
    by_tokens = args.shard == "tokens"
    if by_tokens and cfg.act == "swiglu":
        raise SystemExit("--shard tokens: ReLU modules only")
    layer = rank
    mod, X, W1_0, W2_0, Wg_0 = build_module(cfg, args, dev, layer, by_tokens, world)
    ms_local, launches, clocks, prof, ms_prof, prm, graph_ms = measure(cfg, args, dev, mod, layer, by_tokens, world,
                                                                       args.steps, args.warmup, local_rank,
                                                                       graph=(world == 1 and not args.no_graph))
    ms = parallel.max_over_ranks(ms_local, dev)
    value = (1 if by_tokens else world) * args.steps / (ms * 1e-3)      # one module in all when its tokens are split

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    roofline, roofline_hbm, breakdown = rooflines(cfg, args, prof, args.steps, peaks)

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
        # kept heads: the uniform allocation of the config's sparsity over the heads, rounded by the library
        _, kh = api.sp_allocate_sparsity(torch.ones(1, dtype=torch.float64, device=dev),
                                         torch.tensor([cfg.heads], dtype=torch.int64, device=dev), cfg.sparsity, 1.0,
                                         api.SP_ALLOC_UNIFORM)
        k_heads = max(1, int(kh.item()))
        # results come back into pinned host buffers
        oW1 = torch.empty(cfg.n, cfg.d, dtype=torch.float32).pin_memory(); oW2 = torch.empty(cfg.d, cfg.n, dtype=torch.float32).pin_memory()
        omask = torch.empty(cfg.n, dtype=torch.uint8).pin_memory()
        oWo = torch.empty(cfg.d, cfg.d, dtype=torch.float32).pin_memory(); ohm = torch.empty(cfg.heads, dtype=torch.uint8).pin_memory()
        copy_stream = torch.cuda.Stream(device=dev)

        def prefetch():
            """Starts the host-to-device copies of one layer's inputs on the copy stream; returns (tensors, event)."""
            with torch.cuda.stream(copy_stream):
                bufs = [hX.to(dev, non_blocking=True), hW1.to(dev, non_blocking=True), hW2.to(dev, non_blocking=True),
                        hWg.to(dev, non_blocking=True) if hWg is not None else None,
                        hH.to(dev, non_blocking=True), hWo.to(dev, non_blocking=True)]
                ev = torch.cuda.Event()
                ev.record(copy_stream)
            return bufs, ev

        def one_layer(inputs, start_next: bool):
            """The whole job of one layer from inputs whose copies were started before (a model's layers are streamed:
            while a layer computes, the next one's inputs arrive); starts the next layer's copies when asked.
            Results go to pinned host buffers.  Returns (seconds of the FFN half, seconds in all, next inputs)."""
            t0 = time.perf_counter()
            bufs, ev = inputs
            main = torch.cuda.current_stream()
            main.wait_event(ev)
            for t in bufs:
                if t is not None:
                    t.record_stream(main)
            dX, dW1, dW2, dWg, dH, dWo = bufs
            nxt = prefetch() if start_next else None
            m2 = api.FfnModule(dX, dW1, dW2, dual_mode=args.dual, token_chunk=args.chunk, overlap_k=cfg.k_keep, Wg_0=dWg,
                               pruned_decay=not args.no_pruned_decay)
            m2.sp_ffn_init()
            # this layer's share of pass 0: the importance of the pre-trained module
            api.sp_struct_scores(api.SP_SCORE_WANDA_L2, cfg.n, W=m2.W2_0, colsq=m2.G_A, colsq_stride=cfg.n + 1)
            for _ in range(iters):
                m2.sp_admm_step(prm)
            oW1.copy_(m2.W1, non_blocking=True); oW2.copy_(m2.W2, non_blocking=True); omask.copy_(m2.mask, non_blocking=True)
            torch.cuda.synchronize()
            t_ffn = time.perf_counter()
            # attention module: pre-trained output of the projection, head scores, head mask, W_O recovery on the kept heads
            Ya = torch.empty(dH.shape[0], cfg.d, dtype=dH.dtype, device=dev)
            api.sp_gemm(dH, dWo, Ya, transB=True, use_tensor_cores=(dH.dtype == torch.bfloat16))
            hmask, Wo_new, _ = pipeline.prune_attention_heads(dH, Ya, dWo.float(), cfg.heads, k_heads, rho=cfg.rho,
                                                              token_chunk=args.chunk)
            oWo.copy_(Wo_new, non_blocking=True); ohm.copy_(hmask, non_blocking=True)
            torch.cuda.synchronize()
            t1 = time.perf_counter()
            m2.check_status()
            return t_ffn - t0, t1 - t0, nxt

        # Three layers of a model, streamed.  The first warms the allocator's cache and the library's one-time set-ups
        # and starts the second layer's copies; the timed region covers layers two and three, each of which starts
        # the copies of the layer after it, so it contains two layers' host-to-device copies, compute and results.
        torch.cuda.synchronize()
        t_first0 = time.perf_counter()
        _, _, nxt = one_layer(prefetch(), True)
        torch.cuda.synchronize()
        first_total = time.perf_counter() - t_first0
        t_a = time.perf_counter()
        ffn_a, tot_a, nxt = one_layer(nxt, True)
        ffn_b, tot_b, nxt = one_layer(nxt, True)
        torch.cuda.synchronize()
        copy_stream.synchronize()
        t_total_s = (time.perf_counter() - t_a) / 2.0
        t_ffn_s = 0.5 * (ffn_a + ffn_b)
        t_att_s = 0.5 * ((tot_a - ffn_a) + (tot_b - ffn_b))
        del nxt
        h2d = hX.numel() * hX.element_size() + hW1.numel() * hW1.element_size() + hW2.numel() * hW2.element_size()
        if hWg is not None:
            h2d += hWg.numel() * hWg.element_size()
        h2d += hH.numel() * hH.element_size() + hWo.numel() * hWo.element_size()
        d2h = oW1.numel() * 4 + oW2.numel() * 4 + omask.numel() + oWo.numel() * 4 + ohm.numel()
        e2e = {"value": iters / t_total_s, "unit": UNIT, "layers_per_s": 1.0 / t_total_s, "h2d_bytes_per_step": h2d / iters,
               "d2h_bytes_per_step": d2h / iters, "iterations": iters, "ffn_seconds": t_ffn_s,
               "attention_seconds": t_att_s, "first_layer_seconds": first_total,
               "note": "one pruned layer: pinned-host X, W1_0, W2_0 in; init + importance of the pre-trained module + "
                       "iterations; W1, W2, mask back to host; then the attention half with fixed head outputs (H, "
                       "W_O in; head scores, head mask, W_O recovery on the kept heads; W_O, mask out); "
                       "layers_per_s is that whole job per second, value = iterations / that time; three layers are streamed "
                       "(while a layer computes, the next one's inputs are copied on a second stream), the first is a "
                       "warm-up (first_layer_seconds, its copies not overlapped), the other two are timed together"}
    else:
        del mod, X, W1_0, W2_0, Wg_0
    torch.cuda.empty_cache()

    # ---- the other single-GPU workloads, largest last (one module resident at a time)
    workloads = None
    if args.workloads and world == 1 and not by_tokens:
        workloads = {}
        for name in [w for w in args.workloads.split(",") if w and w != cfg.name]:
            wcfg = synth.CONFIGS[name]
            free, _ = torch.cuda.mem_get_info()
            if free < WORKLOAD_GB.get(name, 0) << 30:
                workloads[name] = {"skipped": f"needs about {WORKLOAD_GB[name]} GB of free device memory"}
                continue
            wmod, wX, wW1, wW2, wWg = build_module(wcfg, args, dev, 0, False, 1)
            w_ms, w_launches, w_clocks, w_prof, w_ms_prof, _, _ = measure(wcfg, args, dev, wmod, 0, False, 1,
                                                                       args.workload_steps, args.workload_warmup,
                                                                       local_rank)
            r_tc, r_hbm, w_break = rooflines(wcfg, args, w_prof, args.workload_steps, peaks)
            workloads[name] = {"workload": workload_name(wcfg), "dtype": DTYPE_NAME[wcfg.storage],
                               "steps": args.workload_steps, "warmup": args.workload_warmup,
                               "ms_per_step": w_ms / args.workload_steps, "value": args.workload_steps / (w_ms * 1e-3),
                               "unit": UNIT, "gpu_launches": w_launches, "clocks": w_clocks, "roofline": r_tc,
                               "roofline_hbm": r_hbm,
                               "solve_phase_ms_per_step": w_break.get("solve_phase", {}).get("ms_per_step"),
                               "profiled_ms_per_step": w_ms_prof / args.workload_steps}
            del wmod, wX, wW1, wW2, wWg
            torch.cuda.empty_cache()

    attention = None
    if world == 1 and not args.no_attention and cfg.storage == "bf16":
        attention = attention_module_timing(cfg, dev)

    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, args.cpu_sample_tokens)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong" if by_tokens else "weak",
            "vs_baseline": None, "dtype": DTYPE_NAME[cfg.storage], "data": "synthetic",
            "config": config_dict(cfg, args, world, by_tokens),
            "clocks": clocks, "gpu_launches": launches, "roofline": roofline, "roofline_hbm": roofline_hbm, "e2e": e2e,
            "cpu_baseline": cpu, "fixed_mask": fixed, "workloads": workloads, "attention_module": attention,
            "profiled_ms_per_step": ms_prof / args.steps, "graph_replay_ms_per_step": graph_ms,
            "profile_note": "value / ms_per_step: timed loop with nothing but the library's launches; roofline, "
                            "roofline_hbm and breakdown: the same steps repeated right after it with a CUDA event pair "
                            "around every launch or phase (profiled_ms_per_step)",
            "breakdown": breakdown}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
