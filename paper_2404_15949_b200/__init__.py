"""B200-native CORM hot path: decode attention over a per-head ragged KV cache fused with recent-message eviction.

``paper_2404_15949_b200.binding`` is the thin ctypes layer over the C-ABI library (same names as ``include/corm.h``);
``paper_2404_15949_b200.workload`` holds the seeded synthetic inputs. Importing the package does not load the CUDA
library; using the binding without a built library raises.
"""
__all__ = ["binding", "workload"]
