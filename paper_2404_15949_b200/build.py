"""In-tree build of the CUDA C-ABI library (sm_100a only) with nvcc."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.environ.get("CORM_LIB_PATH", os.path.join(_HERE, "libcorm.so"))   # override: load another build
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O3", "-lineinfo", "--shared",
              "-Xcompiler", "-fPIC"]


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))) + [
        os.path.join(os.path.dirname(_HERE), "include", "corm.h")]


DEBUG_LIB_PATH = os.path.join(_HERE, "libcorm_dbg.so")


def build_library(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile ``csrc/*.cu`` into ``libcorm.so`` next to this file when it is missing or older than a source.

    ``debug_bounds=True`` builds ``libcorm_dbg.so`` instead, with -DCORM_DEBUG_BOUNDS: every slot, list, record and
    mask index is range-checked in the kernels before use (a failed check sets the device status and skips the
    access). Load it with ``CORM_LIB_PATH=.../libcorm_dbg.so`` and run the GPU tests against it."""
    lib_path = DEBUG_LIB_PATH if debug_bounds else LIB_PATH
    newest = max(os.path.getmtime(s) for s in _sources())
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= newest:
        return lib_path
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-DCORM_DEBUG_BOUNDS"] if debug_bounds else []) + (["-Xptxas", "-v"] if verbose else []) + ["-o", lib_path] + [
        s for s in _sources() if s.endswith(".cu")] + ["-ldl"]      # NVTX (header-only) loads its collector with dlopen
    subprocess.check_call(cmd)
    return lib_path
