"""CPU fp64 oracle for the CORM hot path — TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline leg of ``bench.py`` may import this package.
It shares no code with the CUDA library and never imports it.
"""
from .corm_oracle import CormOracle, build_oracle  # noqa: F401
