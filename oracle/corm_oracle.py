"""ctypes wrapper around ``corm_oracle.c`` (the fp64 CPU oracle) — TEST INFRASTRUCTURE ONLY.

The wrapper only marshals arrays; every arithmetic step lives in the C file, which cites the passages of the paper
(Eq. 1, Eq. 2, Definition 3.1, Definition 4.1, Algorithm 1, the GQA paragraph) it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "corm_oracle.c")
_LIB = os.path.join(_HERE, "libcorm_oracle.so")
_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over units) and return the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build_oracle())
    c_int, c_dbl, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
    lib.oracle_create.restype = vp
    lib.oracle_create.argtypes = [c_int] * 8 + [c_dbl]
    lib.oracle_destroy.argtypes = [vp]
    lib.oracle_decode_step.restype = c_int
    lib.oracle_decode_step.argtypes = [vp, c_int, vp, vp, vp, vp, vp]
    lib.oracle_compress_prompt.restype = c_int
    lib.oracle_compress_prompt.argtypes = [vp, c_int, vp, vp, vp, vp, c_int]
    lib.oracle_live_len.restype = c_int
    lib.oracle_live_len.argtypes = [vp, c_int, c_int, c_int]
    lib.oracle_n_tokens.restype = c_int
    lib.oracle_n_tokens.argtypes = [vp, c_int, c_int]
    lib.oracle_n_obs.restype = c_int
    lib.oracle_n_obs.argtypes = [vp, c_int, c_int]
    lib.oracle_export_unit.restype = c_int
    lib.oracle_export_unit.argtypes = [vp, c_int, c_int, c_int, vp, vp, vp, vp]
    lib.oracle_import_unit.restype = c_int
    lib.oracle_import_unit.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp, vp, vp, c_int, c_int]
    lib.oracle_import_unit_full.restype = c_int
    lib.oracle_import_unit_full.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp, vp, vp, c_int, c_int]
    lib.oracle_export_registers.restype = c_int
    lib.oracle_export_registers.argtypes = [vp, c_int, c_int, c_int, vp]
    lib.oracle_register_words.restype = c_int
    lib.oracle_export_age.restype = c_int
    lib.oracle_export_age.argtypes = [vp, c_int, c_int, c_int, vp]
    lib.oracle_counters.argtypes = [vp, vp, vp, vp, vp]
    lib.oracle_sparsity.argtypes = [vp, vp, vp]
    lib.oracle_sparsity.restype = None
    lib.oracle_similarity.argtypes = [vp, vp, vp]
    lib.oracle_similarity.restype = None
    lib.oracle_set_near_band.argtypes = [vp, c_dbl]
    _lib = lib
    return lib


def _f32(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


class CormOracle:
    """One oracle cache: ``n_layers x batch x n_kv_heads`` units, each an ordered list of live entries.

    Inputs are float32 arrays that carry the cache dtype's values exactly (bf16 and fp32 both embed in float32); the C
    code widens them to double before any arithmetic.
    """

    def __init__(self, n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, window_w, recent_r, alpha):
        self.lib = _load()
        self.L, self.B, self.Hq, self.Hkv = n_layers, batch, n_q_heads, n_kv_heads
        self.d, self.C, self.w, self.r, self.alpha = head_dim, max_tokens, window_w, recent_r, float(alpha)
        self.h = self.lib.oracle_create(n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, window_w,
                                        recent_r, float(alpha))
        if not self.h:
            raise ValueError("oracle_create rejected the configuration")

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.oracle_destroy(self.h)
            self.h = None

    def compress_prompt(self, layer, k_prompt, v_prompt, q_last, prompt_lens):
        prompt_lens = np.ascontiguousarray(prompt_lens, dtype=np.int32)
        assert prompt_lens.shape == (self.B,)
        p_max = int(k_prompt.shape[2]) if k_prompt is not None else 0
        kp = _f32(k_prompt, (self.B, self.Hkv, p_max, self.d)) if p_max else None
        vp = _f32(v_prompt, (self.B, self.Hkv, p_max, self.d)) if p_max else None
        ql = _f32(q_last, (self.B, self.Hq, self.w, self.d)) if p_max else None
        rc = self.lib.oracle_compress_prompt(
            self.h, layer, kp.ctypes.data if p_max else None, vp.ctypes.data if p_max else None,
            ql.ctypes.data if p_max else None, prompt_lens.ctypes.data, p_max)
        if rc:
            raise RuntimeError(f"oracle_compress_prompt failed with code {rc}")

    def decode_step(self, layer, q, k_new, v_new, want_verdicts=False):
        q = _f32(q, (self.B, self.Hq, self.d))
        k_new = _f32(k_new, (self.B, self.Hkv, self.d))
        v_new = _f32(v_new, (self.B, self.Hkv, self.d))
        out = np.empty((self.B, self.Hq, self.d), dtype=np.float64)
        imp = np.zeros((self.B, self.Hkv, self.C), dtype=np.uint8) if want_verdicts else None
        rc = self.lib.oracle_decode_step(self.h, layer, q.ctypes.data, k_new.ctypes.data, v_new.ctypes.data,
                                         out.ctypes.data, imp.ctypes.data if want_verdicts else None)
        if rc:
            raise RuntimeError(f"oracle_decode_step failed with code {rc}")
        return (out, imp) if want_verdicts else out

    def live_len(self, layer, b, h):
        return self.lib.oracle_live_len(self.h, layer, b, h)

    def live_lens(self, layer):
        return np.array([[self.live_len(layer, b, h) for h in range(self.Hkv)] for b in range(self.B)], dtype=np.int32)

    def n_tokens(self, layer, b):
        return self.lib.oracle_n_tokens(self.h, layer, b)

    def n_obs(self, layer, b):
        return self.lib.oracle_n_obs(self.h, layer, b)

    def export_unit(self, layer, b, h):
        l = self.live_len(layer, b, h)
        k = np.empty((l, self.d), dtype=np.float64)
        v = np.empty((l, self.d), dtype=np.float64)
        word = np.empty((l,), dtype=np.uint32)
        pos = np.empty((l,), dtype=np.int32)
        self.lib.oracle_export_unit(self.h, layer, b, h, k.ctypes.data, v.ctypes.data, word.ctypes.data,
                                    pos.ctypes.data)
        age = np.empty((l,), dtype=np.int32)
        self.lib.oracle_export_age(self.h, layer, b, h, age.ctypes.data)
        regs = np.empty((l, self.lib.oracle_register_words()), dtype=np.uint32)       # the whole registers
        self.lib.oracle_export_registers(self.h, layer, b, h, regs.ctypes.data)
        return dict(k=k, v=v, word=word, pos=pos, age=age, regs=regs, live_len=l, n_tokens=self.n_tokens(layer, b),
                    n_obs=self.n_obs(layer, b))

    def import_unit(self, layer, b, h, k, v, word, pos, n_tokens, n_obs):
        """``word``: [live] newest-32-verdict words (windows of up to 32 queries only) or [live, register words]
        whole registers as ``export_unit`` returns them under ``regs`` (any window)."""
        k = np.ascontiguousarray(k, dtype=np.float64)
        v = np.ascontiguousarray(v, dtype=np.float64)
        word = np.ascontiguousarray(word, dtype=np.uint32)
        pos = np.ascontiguousarray(pos, dtype=np.int32)
        if word.ndim == 2:
            assert word.shape == (k.shape[0], self.lib.oracle_register_words())
            fn = self.lib.oracle_import_unit_full
        else:
            assert word.shape == (k.shape[0],)
            fn = self.lib.oracle_import_unit
        rc = fn(self.h, layer, b, h, int(k.shape[0]), k.ctypes.data, v.ctypes.data, word.ctypes.data, pos.ctypes.data,
                int(n_tokens), int(n_obs))
        if rc:
            raise RuntimeError(f"oracle import failed with code {rc}")

    def counters(self):
        vals = [ctypes.c_longlong(0) for _ in range(4)]
        self.lib.oracle_counters(self.h, *[ctypes.byref(x) for x in vals])
        return dict(appended=vals[0].value, evicted=vals[1].value, verdict_evals=vals[2].value,
                    near_threshold=vals[3].value)

    def sparsity(self):
        """(keys judged important, keys judged) over the decode steps so far."""
        a, b = ctypes.c_longlong(0), ctypes.c_longlong(0)
        self.lib.oracle_sparsity(self.h, ctypes.byref(a), ctypes.byref(b))
        return a.value, b.value

    def similarity(self):
        """(sum, count) of Eq. 3 between each query head's query and its query of the previous decode step."""
        a, b = ctypes.c_double(0.0), ctypes.c_longlong(0)
        self.lib.oracle_similarity(self.h, ctypes.byref(a), ctypes.byref(b))
        return a.value, b.value

    def set_near_band(self, rel):
        self.lib.oracle_set_near_band(self.h, float(rel))
