"""B200-native per-module ADMM solver for structured LLM pruning (STRUPRUNE hot path).

`paper_2510_03246_b200.api` is the thin binding over the C-ABI CUDA library `libsp.so`;
`paper_2510_03246_b200.synth` holds the seeded synthetic workload generators.
"""
__all__ = ["api", "synth", "pipeline", "parallel"]
