"""Seeded synthetic workloads (inputs only).

This module produces the tensors both the CUDA library and the CPU oracle consume: queries and keys from AR(1)
chains, planted heavy-hitter keys, iid values, ragged prompt lengths. It holds none of the attention or eviction
arithmetic and imports neither side.
"""
from .generate import (CONFIGS, WorkloadConfig, generate, prompt_lens, n_heavy, heavy_positions,  # noqa: F401
                       build_workload_lib, to_float32_carrier)
