"""Seeded synthetic inputs for the per-module ADMM path (no arithmetic of the method lives here).

The paper calibrates on 128 random 2048-token C4 segments pushed through OPT weights (Section 4.1).
Neither is available offline, so the workloads are replaced by synthetic stand-ins with the same
shapes (Table 1 / Table 3: n = 4 d, 8 d^2 FFN parameters per layer), i.i.d. weights and unit-variance
activations with a few outlier input channels.

Everything is a pure function of (seed, tensor id, element index): a counter-based integer hash
gives 32 uniform bits per element, which are turned into Gaussian / Laplace variates.  The same
code runs on CPU tensors (for the CPU oracle) and on CUDA tensors (for the benchmark); the integer
stream is bit-identical on both, the float transforms may differ in the last ulp, so parity tests
always hand ONE generated array to both sides.
"""
from __future__ import annotations

import dataclasses
import math

import torch

BASE_SEED = 2510032460
_M32 = 0xFFFFFFFF


@dataclasses.dataclass(frozen=True)
class ModuleConfig:
    """Shape and distribution of one FFN module workload."""

    name: str
    layers: int
    d: int  # d_model
    n: int  # FFN hidden channels
    heads: int
    d_head: int
    tokens: int  # N = sequences x tokens per sequence
    storage: str  # "f32" or "bf16"
    weight_std: float
    act_dist: str  # "gauss" or "laplace"
    outlier_frac: float
    outlier_scale: float
    sparsity: float
    iters: int
    rho: float
    act: str = "relu"
    cfg_id: int = 0

    @property
    def k_keep(self) -> int:
        return self.n - int(math.floor(self.sparsity * self.n + 0.5))


CONFIGS = {
    "C1": ModuleConfig("C1", 2, 768, 3072, 12, 64, 16 * 128, "f32", 0.02, "gauss", 0.01, 20.0, 0.5, 10, 0.1, cfg_id=1),
    "C2": ModuleConfig("C2", 24, 2048, 8192, 32, 64, 128 * 2048, "bf16", 0.02, "gauss", 0.005, 30.0, 0.5, 20, 0.1, cfg_id=2),
    "C3": ModuleConfig("C3", 32, 4096, 16384, 32, 128, 128 * 2048, "bf16", 0.015, "laplace", 0.005, 40.0, 0.6, 20, 0.1, cfg_id=3),
    "C4": ModuleConfig("C4", 32, 4096, 11008, 32, 128, 128 * 4096, "bf16", 0.02, "gauss", 0.01, 50.0, 0.7, 30, 0.1, act="swiglu", cfg_id=4),
    "C5": ModuleConfig("C5", 1, 7168, 28672, 56, 128, 256 * 2048, "bf16", 0.01, "gauss", 0.01, 30.0, 0.8, 50, 0.1, cfg_id=5),
}


def scaled(cfg: ModuleConfig, **kw) -> ModuleConfig:
    """A copy of `cfg` with some fields replaced (token-reduced or width-reduced test cases)."""
    return dataclasses.replace(cfg, **kw)


def module_seed(cfg: ModuleConfig, layer: int = 0) -> int:
    return BASE_SEED + 100 * cfg.cfg_id + layer


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """A 32-bit avalanche mixer (xorshift-multiply rounds) evaluated in int64 lanes."""
    x = x & _M32
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def uniform_bits(seed: int, tensor_id: int, start: int, count: int, device="cpu", stream: int = 0) -> torch.Tensor:
    """32 random bits (as int64 in [0, 2^32)) for elements start..start+count-1 of tensor `tensor_id`."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    lo = idx & _M32
    hi = (idx >> 32) & _M32
    key = (seed * 0x9E3779B1 + tensor_id * 0x85EBCA77 + stream * 0xC2B2AE3D + 0x27D4EB2F) & _M32
    h = _mix32(lo ^ key)
    h = _mix32(h + hi * 0x165667B1 + (key >> 7))
    return h


def _unit_open(bits: torch.Tensor) -> torch.Tensor:
    """Map 32 bits to a double in (0, 1)."""
    return (bits.to(torch.float64) + 0.5) * (1.0 / 4294967296.0)


def standard_variates(seed: int, tensor_id: int, numel: int, dist: str, device="cpu",
                      chunk: int = 1 << 24) -> torch.Tensor:
    """`numel` unit-variance variates (float32) of the named distribution, generated chunk by chunk."""
    out = torch.empty(numel, dtype=torch.float32, device=device)
    for s in range(0, numel, chunk):
        c = min(chunk, numel - s)
        u1 = _unit_open(uniform_bits(seed, tensor_id, s, c, device, stream=0))
        u2 = _unit_open(uniform_bits(seed, tensor_id, s, c, device, stream=1))
        if dist == "gauss":
            v = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        elif dist == "laplace":
            # inverse CDF of a Laplace variate scaled to unit variance (scale b = 1/sqrt 2)
            sign = torch.where(u2 < 0.5, -1.0, 1.0)
            v = -sign * torch.log(u1) * (1.0 / math.sqrt(2.0))
        else:
            raise ValueError(f"unknown distribution {dist!r}")
        out[s:s + c] = v.to(torch.float32)
    return out


def outlier_channels(seed: int, tensor_id: int, channels: int, frac: float) -> torch.Tensor:
    """Indices of the ceil(frac*channels) channels that carry the outlier scale (seeded, sorted)."""
    m = int(math.ceil(frac * channels)) if frac > 0 else 0
    if m == 0:
        return torch.empty(0, dtype=torch.int64)
    bits = uniform_bits(seed, tensor_id, 0, channels, "cpu", stream=7)
    order = torch.argsort(bits * channels + torch.arange(channels), stable=True)
    return torch.sort(order[:m]).values


def storage_dtype(cfg: ModuleConfig) -> torch.dtype:
    return torch.float32 if cfg.storage == "f32" else torch.bfloat16


def make_activations(cfg: ModuleConfig, layer: int = 0, device="cpu", tokens: int | None = None,
                     tensor_id: int = 1) -> torch.Tensor:
    """Module input X as a token-major [N, d] tensor in the config's storage dtype."""
    N = cfg.tokens if tokens is None else tokens
    seed = module_seed(cfg, layer)
    x = standard_variates(seed, tensor_id, N * cfg.d, cfg.act_dist, device).view(N, cfg.d)
    ch = outlier_channels(seed, tensor_id, cfg.d, cfg.outlier_frac).to(device)
    if ch.numel():
        x[:, ch] *= cfg.outlier_scale
    return x.to(storage_dtype(cfg))


def make_weights(cfg: ModuleConfig, layer: int = 0, device="cpu"):
    """Pre-trained stand-ins W1_0 [n, d] (up-projection) and W2_0 [d, n] (down-projection), storage dtype."""
    seed = module_seed(cfg, layer)
    w1 = standard_variates(seed, 2, cfg.n * cfg.d, "gauss", device).view(cfg.n, cfg.d) * cfg.weight_std
    w2 = standard_variates(seed, 3, cfg.d * cfg.n, "gauss", device).view(cfg.d, cfg.n) * cfg.weight_std
    dt = storage_dtype(cfg)
    return w1.to(dt), w2.to(dt)


def make_gate_weights(cfg: ModuleConfig, layer: int = 0, device="cpu"):
    """Pre-trained stand-in of the gate projection Wg_0 [n, d] of a SwiGLU module (tensor id 4), storage dtype."""
    seed = module_seed(cfg, layer)
    wg = standard_variates(seed, 4, cfg.n * cfg.d, "gauss", device).view(cfg.n, cfg.d) * cfg.weight_std
    return wg.to(storage_dtype(cfg))


def make_attention_inputs(cfg: ModuleConfig, layer: int = 0, device="cpu", tokens: int | None = None):
    """Stand-ins for one attention module with its head outputs held fixed: the concatenated head outputs H [N, d]
    (drawn like the module input, tensor id 5) and the output projection W_O [d, d] (tensor id 6, storage dtype)."""
    H = make_activations(cfg, layer, device, tokens, tensor_id=5)
    wo = standard_variates(module_seed(cfg, layer), 6, cfg.d * cfg.d, "gauss", device).view(cfg.d, cfg.d) * cfg.weight_std
    return H, wo.to(storage_dtype(cfg))


def make_importances(cfg: ModuleConfig, device="cpu") -> torch.Tensor:
    """A seeded stand-in for the per-layer importances I_l (float64, positive, mildly depth dependent)."""
    u = _unit_open(uniform_bits(module_seed(cfg, 0), 9, 0, cfg.layers, device))
    depth = torch.arange(cfg.layers, dtype=torch.float64, device=device) / max(cfg.layers - 1, 1)
    return (1.0 + 0.5 * u) * (1.0 - 0.3 * depth)
