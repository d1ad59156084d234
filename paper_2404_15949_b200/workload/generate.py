"""Assembly of the synthetic workloads from the counter-based noise in ``gen.c``.

Recipe (one layer; every tensor is rounded once to the cache dtype and carried as float32):
  keys     one AR(1) chain (rho 0.9, sigma 0.44) per (layer, sequence, kv head) over token positions 1..P+steps;
           at H planted positions in [1, P-r] the key is replaced by 4*u, u ~ N(0, I) ("heavy hitters");
           optional drift: from decode step ``drift_every`` on, the first ``drift_count`` keys of every block of
           ``drift_every`` steps are planted the same way.
  values   iid N(0, 1).
  queries  one AR(1) chain per (layer, sequence, query head); with grouped queries the heads of a group mix a chain
           shared by the group (weight sqrt(gqa_rho)) with a private one (weight sqrt(1 - gqa_rho)).
           Chain index 0 sits at prompt position max(1, P-w+1), so ``q_last`` holds the last w prompt queries.
  lengths  P_b = prompt_min + hash mod (prompt_max - prompt_min + 1).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libcorm_workload.so")
_lib = None

T_KEY, T_VALUE, T_QUERY, T_QUERY_SHARED, T_HH_DIR, T_HH_POS, T_HH_COUNT, T_PROMPT_LEN = range(1, 9)


def build_workload_lib(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_workload_lib())
        u64, u32, i64, i32, dbl, vp = (ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int64, ctypes.c_int32,
                                       ctypes.c_double, ctypes.c_void_p)
        lib.wl_uniform_u64.restype = u64
        lib.wl_uniform_u64.argtypes = [u64, u32, u32, u32, u32, u64]
        lib.wl_normal_block.argtypes = [u64, u32, u32, u32, u32, u64, i64, i32, vp]
        lib.wl_ar1_chain.argtypes = [u64, u32, u32, u32, u32, i64, i32, dbl, dbl, vp]
        lib.wl_round_bf16.argtypes = [vp, i64]
        _lib = lib
    return _lib


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str            # "f32" or "bf16": dtype of the cache, q, k_new, v_new, out
    prompt_min: int
    prompt_max: int
    steps: int
    window_w: int
    recent_r: int
    alpha: float
    hh_min: int           # planted heavy hitters per unit: uniform in [hh_min, hh_max]
    hh_max: int
    dense_layers: int = 0  # the first `dense_layers` layers get no heavy hitters
    gqa_rho: float = 0.0   # pairwise correlation of query heads inside a group
    drift_every: int = 0
    drift_count: int = 0
    rho: float = 0.9
    sigma: float = 0.44
    hh_scale: float = 4.0
    seed: int = 15949

    @property
    def max_tokens(self) -> int:
        return self.prompt_max + self.steps

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def with_(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


# The five benchmark configurations (shapes and parameters of the synthetic stand-ins).
CONFIGS = {
    1: WorkloadConfig("tiny_f32", 1, 1, 8, 8, 128, "f32", 512, 512, 64, 8, 32, 1.0, 4, 4),
    2: WorkloadConfig("llama2_7b_bf16", 32, 1, 32, 32, 128, "bf16", 4096, 4096, 256, 8, 256, 1.0, 8, 64,
                      dense_layers=3),
    3: WorkloadConfig("batch32_bf16", 1, 32, 32, 32, 128, "bf16", 2048, 4096, 512, 8, 256, 1.0, 8, 64),
    4: WorkloadConfig("gqa_llama3_8b_bf16", 1, 16, 32, 8, 128, "bf16", 8192, 8192, 256, 8, 256, 1.0, 8, 64,
                      gqa_rho=0.7),
    5: WorkloadConfig("long_gqa_bf16", 1, 4, 32, 8, 128, "bf16", 32768, 32768, 1024, 16, 512, 1.0, 16, 16,
                      gqa_rho=0.7, drift_every=128, drift_count=4),
}


def to_float32_carrier(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float32 array once to the cache dtype (ties to even), in place when possible; stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        _load().wl_round_bf16(a.ctypes.data, a.size)
    elif dtype != "f32":
        raise ValueError(dtype)
    return a


def prompt_lens(cfg: WorkloadConfig) -> np.ndarray:
    lib = _load()
    span = cfg.prompt_max - cfg.prompt_min + 1
    return np.array([cfg.prompt_min + lib.wl_uniform_u64(cfg.seed, T_PROMPT_LEN, 0, b, 0, 0) % span
                     for b in range(cfg.batch)], dtype=np.int32)


def n_heavy(cfg: WorkloadConfig, layer: int, seq: int, head: int) -> int:
    if layer < cfg.dense_layers:
        return 0
    span = cfg.hh_max - cfg.hh_min + 1
    return cfg.hh_min + int(_load().wl_uniform_u64(cfg.seed, T_HH_COUNT, layer, seq, head, 0) % span)


def heavy_positions(cfg: WorkloadConfig, layer: int, seq: int, head: int, P: int) -> np.ndarray:
    """Planted prompt positions (1-based, unique, sorted) of one unit: H draws uniform in [1, P-r]."""
    hi = P - cfg.recent_r
    if hi < 1:
        return np.zeros((0,), dtype=np.int64)
    lib = _load()
    H = n_heavy(cfg, layer, seq, head)
    return np.unique(np.array([1 + lib.wl_uniform_u64(cfg.seed, T_HH_POS, layer, seq, head, i) % hi
                               for i in range(H)], dtype=np.int64))


def _drift_steps(cfg: WorkloadConfig, n_steps: int) -> list:
    if not cfg.drift_every:
        return []
    return [s for s in range(1, n_steps + 1) if s >= cfg.drift_every and s % cfg.drift_every < cfg.drift_count]


def _key_chain(cfg, layer, seq, head, P, n_steps):
    lib = _load()
    n, d = P + n_steps, cfg.head_dim
    out = np.empty((n, d), dtype=np.float32)
    if n:
        lib.wl_ar1_chain(cfg.seed, T_KEY, layer, seq, head, n, d, cfg.rho, cfg.sigma, out.ctypes.data)
    planted = [int(p) for p in heavy_positions(cfg, layer, seq, head, P)] + [P + s for s in _drift_steps(cfg, n_steps)]
    u = np.empty((1, d), dtype=np.float32)
    for p in planted:
        lib.wl_normal_block(cfg.seed, T_HH_DIR, layer, seq, head, p, 1, d, u.ctypes.data)
        out[p - 1] = np.float32(cfg.hh_scale) * u[0]
    return out


def _value_rows(cfg, layer, seq, head, n):
    out = np.empty((n, cfg.head_dim), dtype=np.float32)
    if n:
        _load().wl_normal_block(cfg.seed, T_VALUE, layer, seq, head, 0, n, cfg.head_dim, out.ctypes.data)
    return out


def _ar1(cfg, tensor, layer, seq, head, n):
    out = np.empty((n, cfg.head_dim), dtype=np.float32)
    if n:
        _load().wl_ar1_chain(cfg.seed, tensor, layer, seq, head, n, cfg.head_dim, cfg.rho, cfg.sigma,
                             out.ctypes.data)
    return out


def generate(cfg: WorkloadConfig, layer: int = 0, seqs=None, kv_heads=None, n_steps=None, threads=None):
    """Inputs of one layer for the chosen sequences and kv heads (defaults: all), prompt plus ``n_steps`` decode steps.

    Returns a namespace of float32 arrays whose values are exactly representable in ``cfg.dtype``:
      prompt_lens [nb] int32, k_prompt/v_prompt [nb, nh, p_max, d] (rows past a sequence's length are zero),
      q_last [nb, nh*G, w, d], q [n_steps, nb, nh*G, d], k_new/v_new [n_steps, nb, nh, d].
    Slices are independent of which other sequences/heads are requested.
    """
    seqs = list(range(cfg.batch)) if seqs is None else list(seqs)
    kv_heads = list(range(cfg.n_kv_heads)) if kv_heads is None else list(kv_heads)
    n_steps = cfg.steps if n_steps is None else int(n_steps)
    G, d, w = cfg.group, cfg.head_dim, cfg.window_w
    all_lens = prompt_lens(cfg)
    lens = all_lens[seqs]
    nb, nh = len(seqs), len(kv_heads)
    p_max = int(lens.max()) if nb else 0
    k_prompt = np.zeros((nb, nh, p_max, d), dtype=np.float32)
    v_prompt = np.zeros((nb, nh, p_max, d), dtype=np.float32)
    q_last = np.zeros((nb, nh * G, w, d), dtype=np.float32)
    q = np.zeros((n_steps, nb, nh * G, d), dtype=np.float32)
    k_new = np.zeros((n_steps, nb, nh, d), dtype=np.float32)
    v_new = np.zeros((n_steps, nb, nh, d), dtype=np.float32)
    mix_shared, mix_private = np.float32(np.sqrt(cfg.gqa_rho)), np.float32(np.sqrt(1.0 - cfg.gqa_rho))

    def unit(job):
        ib, ih = job
        b, h, P = seqs[ib], kv_heads[ih], int(lens[ib])
        keys = _key_chain(cfg, layer, b, h, P, n_steps)
        vals = _value_rows(cfg, layer, b, h, P + n_steps)
        k_prompt[ib, ih, :P] = keys[:P]
        v_prompt[ib, ih, :P] = vals[:P]
        k_new[:, ib, ih] = keys[P:]
        v_new[:, ib, ih] = vals[P:]
        wp = min(P, w)
        nq = wp + n_steps
        shared = _ar1(cfg, T_QUERY_SHARED, layer, b, h, nq) if cfg.gqa_rho > 0 else None
        for g in range(G):
            qh = h * G + g
            chain = _ar1(cfg, T_QUERY, layer, b, qh, nq)
            if shared is not None:
                chain = mix_shared * shared + mix_private * chain
            q_last[ib, ih * G + g, w - wp:] = chain[:wp]
            q[:, ib, ih * G + g] = chain[wp:]

    jobs = [(ib, ih) for ib in range(nb) for ih in range(nh)]
    threads = threads or min(32, os.cpu_count() or 1)
    if len(jobs) > 1 and threads > 1:
        with ThreadPoolExecutor(threads) as pool:
            list(pool.map(unit, jobs))
    else:
        for job in jobs:
            unit(job)
    for a in (k_prompt, v_prompt, q_last, q, k_new, v_new):
        to_float32_carrier(a, cfg.dtype)
    return SimpleNamespace(cfg=cfg, layer=layer, seqs=seqs, kv_heads=kv_heads, n_steps=n_steps, prompt_lens=lens,
                           k_prompt=k_prompt, v_prompt=v_prompt, q_last=q_last, q=q, k_new=k_new, v_new=v_new)
