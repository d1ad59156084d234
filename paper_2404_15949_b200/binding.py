"""Thin ctypes binding over ``libcorm.so`` — argument marshalling only, same names as ``include/corm.h``.

PyTorch supplies device memory (the arena and the tensors) and the CUDA stream; every step of the path runs inside
the library's kernels. There is no CPU fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

from .build import LIB_PATH

CORM_OK = 0
CORM_F32, CORM_BF16 = 0, 1
STATUS_NAMES = {0: "CORM_OK", 1: "CORM_ERR_INVALID_ARG", 2: "CORM_ERR_UNSUPPORTED", 3: "CORM_ERR_ARENA_TOO_SMALL",
                4: "CORM_ERR_STATE", 5: "CORM_ERR_CUDA", 6: "CORM_ERR_CAPACITY", 7: "CORM_ERR_TIMEOUT"}


class CormConfig(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("max_tokens", ctypes.c_int32),
                ("window_w", ctypes.c_int32), ("recent_r", ctypes.c_int32), ("alpha", ctypes.c_float),
                ("kv_dtype", ctypes.c_int32), ("device", ctypes.c_int32)]


class CormStats(ctypes.Structure):
    _fields_ = [("live_keys", ctypes.c_int64), ("appended_keys", ctypes.c_int64), ("evicted_keys", ctypes.c_int64),
                ("retention", ctypes.c_double), ("kv_bytes_live", ctypes.c_int64), ("aux_bytes_live", ctypes.c_int64),
                ("moved_rows", ctypes.c_int64), ("attended_keys", ctypes.c_int64), ("device_status", ctypes.c_int32),
                ("important_keys", ctypes.c_int64), ("near_threshold", ctypes.c_int64)]


class CormError(RuntimeError):
    def __init__(self, call, status):
        self.status = status
        super().__init__(f"{call} -> {STATUS_NAMES.get(status, status)}")


_lib = None


def load_library():
    """dlopen the in-tree library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run paper_2404_15949_b200.build.build_library() "
                           "(or __graft_entry__.build()) first; the CORM path has no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(CormConfig)
    lib.corm_cache_arena_bytes.restype = sz
    lib.corm_cache_arena_bytes.argtypes = [cfgp]
    lib.corm_cache_create.restype = i32
    lib.corm_cache_create.argtypes = [cfgp, vp, sz, ctypes.POINTER(vp)]
    lib.corm_cache_arena_bytes_paged.restype = sz
    lib.corm_cache_arena_bytes_paged.argtypes = [cfgp, i32]
    lib.corm_cache_create_paged.restype = i32
    lib.corm_cache_create_paged.argtypes = [cfgp, i32, vp, sz, ctypes.POINTER(vp)]
    lib.corm_cache_pool_usage.restype = i32
    lib.corm_cache_pool_usage.argtypes = [vp, i32, vp, vp, vp]
    lib.corm_cache_destroy.restype = i32
    lib.corm_cache_destroy.argtypes = [vp]
    lib.corm_cache_reset.restype = i32
    lib.corm_cache_reset.argtypes = [vp, vp]
    lib.corm_compress_prompt.restype = i32
    lib.corm_compress_prompt.argtypes = [vp, i32, vp, vp, vp, vp, i32, vp]
    lib.corm_decode_step.restype = i32
    lib.corm_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.corm_decode_step_static.restype = i32
    lib.corm_decode_step_static.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.corm_decode_step_host.restype = i32
    lib.corm_decode_step_host.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.corm_decode_step_layers.restype = i32
    lib.corm_decode_step_layers.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.corm_decode_steps.restype = i32
    lib.corm_decode_steps.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.corm_decode_steps_host.restype = i32
    lib.corm_decode_steps_host.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.corm_cache_chained_launches.restype = i64
    lib.corm_cache_chained_launches.argtypes = [vp]
    lib.corm_cache_stats.restype = i32
    lib.corm_cache_stats.argtypes = [vp, ctypes.POINTER(CormStats), vp]
    lib.corm_cache_live_lens.restype = i32
    lib.corm_cache_live_lens.argtypes = [vp, i32, vp, vp]
    lib.corm_cache_export_state.restype = i32
    lib.corm_cache_export_state.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.corm_cache_import_state.restype = i32
    lib.corm_cache_import_state.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, i32, i32, i32, vp]
    lib.corm_cache_set_tuning.restype = i32
    lib.corm_cache_set_tuning.argtypes = [vp, i32, i32]
    lib.corm_cache_set_similarity_monitor.restype = ctypes.c_int
    lib.corm_cache_set_similarity_monitor.argtypes = [vp, ctypes.c_int32]
    lib.corm_cache_similarity.restype = ctypes.c_int
    lib.corm_cache_similarity.argtypes = [vp, vp, vp, vp]
    lib.corm_cache_set_bound_scale.restype = ctypes.c_int
    lib.corm_cache_set_bound_scale.argtypes = [vp, ctypes.c_double]
    lib.corm_cache_kernel_launches.restype = i64
    lib.corm_cache_kernel_launches.argtypes = [vp]
    lib.corm_status_string.restype = ctypes.c_char_p
    lib.corm_status_string.argtypes = [i32]
    _lib = lib
    return lib


def _check(call, rc):
    if rc != CORM_OK:
        raise CormError(call, rc)


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _torch_dtype(kv_dtype):
    return torch.bfloat16 if kv_dtype == CORM_BF16 else torch.float32


def _np_view_dtype(kv_dtype):
    return np.uint16 if kv_dtype == CORM_BF16 else np.float32


def corm_cache_arena_bytes(cfg: CormConfig) -> int:
    return int(load_library().corm_cache_arena_bytes(ctypes.byref(cfg)))


class CormCache:
    """Owns the arena tensor (torch device memory) and the library's host object."""

    def __init__(self, n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, window_w, recent_r, alpha,
                 kv_dtype="bf16", device=0, pool_pages=0):
        """pool_pages = 0: one slab of max_tokens rows per unit; > 0: a paged cache with that many 32-key pages of K
        and of V per layer (corm_cache_create_paged)."""
        self.lib = load_library()
        code = {"bf16": CORM_BF16, "f32": CORM_F32}[kv_dtype]
        self.cfg = CormConfig(n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, window_w, recent_r,
                              float(alpha), code, device)
        self._q_shape = (batch, n_q_heads, head_dim)
        self._kv_shape = (batch, n_kv_heads, head_dim)
        self.kv_dtype, self.dtype, self.device = code, _torch_dtype(code), torch.device("cuda", device)
        self.pool_pages = int(pool_pages)
        nbytes = int(self.lib.corm_cache_arena_bytes_paged(ctypes.byref(self.cfg), self.pool_pages))
        if nbytes == 0:
            raise CormError("corm_cache_arena_bytes_paged", 1)
        self.arena = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        handle = ctypes.c_void_p()
        _check("corm_cache_create_paged", self.lib.corm_cache_create_paged(
            ctypes.byref(self.cfg), self.pool_pages, self.arena.data_ptr(), nbytes, ctypes.byref(handle)))
        self.handle = handle

    def close(self):
        if getattr(self, "handle", None):
            self.lib.corm_cache_destroy(self.handle)
            self.handle = None

    __del__ = close

    # ---- the four calls of the boundary -------------------------------------------------------------------------
    def corm_compress_prompt(self, layer, k_prompt, v_prompt, q_last, prompt_lens, stream=None):
        lens = np.ascontiguousarray(prompt_lens, dtype=np.int32)
        assert lens.shape == (self.cfg.batch,)
        p_max = int(k_prompt.shape[2]) if k_prompt is not None else 0
        for t in (k_prompt, v_prompt, q_last):
            assert t is None or (t.is_cuda and t.is_contiguous() and t.dtype == self.dtype)
        if p_max:
            assert tuple(k_prompt.shape) == (self.cfg.batch, self.cfg.n_kv_heads, p_max, self.cfg.head_dim)
            assert tuple(v_prompt.shape) == tuple(k_prompt.shape)
            assert tuple(q_last.shape) == (self.cfg.batch, self.cfg.n_q_heads, self.cfg.window_w, self.cfg.head_dim)
        ptr = lambda t: t.data_ptr() if (t is not None and t.numel()) else None
        _check("corm_compress_prompt", self.lib.corm_compress_prompt(
            self.handle, layer, ptr(k_prompt), ptr(v_prompt), ptr(q_last), lens.ctypes.data, p_max,
            _stream_ptr(stream)))

    def _check_step_args(self, call, q, k_new, v_new, out):
        # kept cheap: these calls are on the per-token path and a launch is only a few microseconds
        if q.shape != self._q_shape or k_new.shape != self._kv_shape or v_new.shape != self._kv_shape:
            raise ValueError(f"{call}: q / k_new / v_new have the wrong shape")
        if not (q.dtype == k_new.dtype == v_new.dtype == self.dtype and q.is_cuda and k_new.is_cuda and v_new.is_cuda
                and q.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous()):
            raise ValueError(f"{call}: inputs must be contiguous device tensors of the cache dtype")
        if out is not None and not (out.shape == self._q_shape and out.dtype == self.dtype and out.is_cuda
                                    and out.is_contiguous()):
            raise ValueError(f"{call}: out must be a contiguous device tensor shaped like q")

    def corm_decode_step(self, layer, q, k_new, v_new, out=None, stream=None):
        self._check_step_args("corm_decode_step", q, k_new, v_new, out)
        if out is None:
            out = torch.empty_like(q)
        rc = self.lib.corm_decode_step(self.handle, layer, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                                       out.data_ptr(), _stream_ptr(stream))
        if rc != CORM_OK:
            raise CormError("corm_decode_step", rc)
        return out

    def corm_decode_step_layers(self, first_layer, q, k_new, v_new, out, stream=None):
        """One decode step of ``len(q)`` consecutive layers from a single host call. ``q``, ``k_new``, ``v_new``,
        ``out``: sequences of per-layer tensors, or ``numpy`` uint64 arrays of their device addresses as
        ``pointer_table`` builds them (no per-tensor work on the host then; shapes were checked when it was built)."""
        n = len(q)
        if not (len(k_new) == len(v_new) == len(out) == n and n >= 1):
            raise ValueError("corm_decode_step_layers: one q, k_new, v_new and out per layer")
        tables = []
        for i, ts in enumerate((q, k_new, v_new, out)):
            if isinstance(ts, np.ndarray):
                assert ts.dtype == np.uint64 and ts.flags.c_contiguous
                tables.append(ts)
            else:
                tables.append(self.pointer_table(ts, "q" if i in (0, 3) else "kv"))
        _check("corm_decode_step_layers", self.lib.corm_decode_step_layers(
            self.handle, first_layer, n, tables[0].ctypes.data, tables[1].ctypes.data, tables[2].ctypes.data,
            tables[3].ctypes.data, _stream_ptr(stream)))
        return out

    def corm_decode_steps(self, first_layer, n_layers, q, k_new, v_new, out=None, stream=None):
        """``q.shape[0]`` consecutive decode steps of ``n_layers`` consecutive layers from one host call. ``q`` and
        ``out``: device tensors ``[n_steps, n_layers, batch, n_q_heads, head_dim]``; ``k_new``, ``v_new``:
        ``[n_steps, n_layers, batch, n_kv_heads, head_dim]`` (the layer axis may be left out for one layer)."""
        if n_layers == 1 and q.dim() == 1 + len(self._q_shape):
            q, k_new, v_new = q.unsqueeze(1), k_new.unsqueeze(1), v_new.unsqueeze(1)
            out = out.unsqueeze(1) if out is not None else None
            squeeze = True
        else:
            squeeze = False
        n_steps = q.shape[0]
        if out is None:
            out = torch.empty_like(q)
        for t, shape in ((q, self._q_shape), (out, self._q_shape), (k_new, self._kv_shape), (v_new, self._kv_shape)):
            if not (tuple(t.shape) == (n_steps, n_layers) + tuple(shape) and t.dtype == self.dtype and t.is_cuda and
                    t.is_contiguous()):
                raise ValueError("corm_decode_steps: contiguous device tensors [n_steps, n_layers, ...] of the cache dtype")
        _check("corm_decode_steps", self.lib.corm_decode_steps(
            self.handle, first_layer, n_layers, n_steps, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
            _stream_ptr(stream)))
        return out.squeeze(1) if squeeze else out

    def corm_decode_steps_host(self, first_layer, n_layers, q, k_new, v_new, out, stream=None):
        """corm_decode_steps on host tensors ``[n_steps, n_layers, ...]`` (pinned ones are used in place)."""
        n_steps = q.shape[0]
        for t, shape in ((q, self._q_shape), (out, self._q_shape), (k_new, self._kv_shape), (v_new, self._kv_shape)):
            if not (tuple(t.shape) == (n_steps, n_layers) + tuple(shape) and t.dtype == self.dtype and not t.is_cuda and
                    t.is_contiguous()):
                raise ValueError("corm_decode_steps_host: contiguous host tensors [n_steps, n_layers, ...] of the cache dtype")
        _check("corm_decode_steps_host", self.lib.corm_decode_steps_host(
            self.handle, first_layer, n_layers, n_steps, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
            _stream_ptr(stream)))
        return out

    def corm_cache_chained_launches(self):
        return int(self.lib.corm_cache_chained_launches(self.handle))

    def pointer_table(self, tensors, kind):
        """Device addresses of per-layer tensors as a uint64 array (kind "q": shaped like q / out, "kv": like k_new)."""
        shape = self._q_shape if kind == "q" else self._kv_shape
        for t in tensors:
            if not (t.shape == shape and t.dtype == self.dtype and t.is_cuda and t.is_contiguous()):
                raise ValueError("pointer_table: contiguous device tensors of the cache dtype with the step's shape")
        return np.array([t.data_ptr() for t in tensors], dtype=np.uint64)

    def corm_decode_step_static(self, layer, q, k_new, v_new, out=None, stream=None):
        """corm_decode_step for callers that must not allocate: the step's scratch sits in an array built into the
        library (16 MiB, shared by every cache on the device) instead of the arena. Pass ``out`` to keep this
        wrapper allocation-free as well; calls that overlap on the GPU race on the shared array."""
        self._check_step_args("corm_decode_step_static", q, k_new, v_new, out)
        if out is None:
            out = torch.empty_like(q)
        _check("corm_decode_step_static", self.lib.corm_decode_step_static(
            self.handle, layer, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(), _stream_ptr(stream)))
        return out

    def corm_decode_step_host(self, layer, q, k_new, v_new, out, stream=None):
        """Host (pinned) tensors in and out; the copies run inside the library on the same stream."""
        for t in (q, k_new, v_new, out):
            assert not t.is_cuda and t.is_contiguous() and t.dtype == self.dtype
        _check("corm_decode_step_host", self.lib.corm_decode_step_host(
            self.handle, layer, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(), _stream_ptr(stream)))
        return out

    def corm_cache_stats(self, stream=None):
        st = CormStats()
        _check("corm_cache_stats", self.lib.corm_cache_stats(self.handle, ctypes.byref(st), _stream_ptr(stream)))
        return {name: getattr(st, name) for name, _ in CormStats._fields_}

    # ---- helpers --------------------------------------------------------------------------------------------------
    def corm_cache_pool_usage(self, layer=0, stream=None):
        """(pages in use, pages in total) of one layer's pool; (0, 0) for a slab cache."""
        used, total = ctypes.c_int64(0), ctypes.c_int64(0)
        _check("corm_cache_pool_usage", self.lib.corm_cache_pool_usage(self.handle, layer, ctypes.byref(used),
                                                                       ctypes.byref(total), _stream_ptr(stream)))
        return int(used.value), int(total.value)

    def corm_cache_reset(self, stream=None):
        _check("corm_cache_reset", self.lib.corm_cache_reset(self.handle, _stream_ptr(stream)))

    def corm_cache_live_lens(self, layer, stream=None):
        out = np.empty((self.cfg.batch, self.cfg.n_kv_heads), dtype=np.int32)
        _check("corm_cache_live_lens", self.lib.corm_cache_live_lens(self.handle, layer, out.ctypes.data,
                                                                     _stream_ptr(stream)))
        return out

    def corm_cache_set_tuning(self, split_len=0, allow_fast_path=True):
        """allow_fast_path: False/0 generic kernels, True/1 automatic, 2 / 3 block-per-split kernels that always finish
        units of several splits inside the decode launch / by the verdict launch, 4 / 5 the balanced kernel finishing
        inside its launch / with the verdict launch, 6 that kernel's loop with a block per split and each unit finished
        by its last split."""
        _check("corm_cache_set_tuning", self.lib.corm_cache_set_tuning(self.handle, split_len, int(allow_fast_path)))

    def corm_cache_set_similarity_monitor(self, enabled=True):
        _check("corm_cache_set_similarity_monitor", self.lib.corm_cache_set_similarity_monitor(self.handle, int(enabled)))

    def corm_cache_similarity(self, stream=None):
        """(sum, count) of the adjacent-query cosine similarities (Eq. 3) recorded while the monitor was on."""
        total, n = ctypes.c_double(0.0), ctypes.c_int64(0)
        _check("corm_cache_similarity", self.lib.corm_cache_similarity(self.handle, ctypes.byref(total), ctypes.byref(n),
                                                                     _stream_ptr(stream)))
        return total.value, n.value

    def corm_cache_set_bound_scale(self, scale):
        """Multiplies the proven fp32 error bound of the tiled prompt pass (>= 1; results never change, only how many
        logits are formed again in fp64)."""
        _check("corm_cache_set_bound_scale", self.lib.corm_cache_set_bound_scale(self.handle, float(scale)))

    def corm_cache_kernel_launches(self):
        return int(self.lib.corm_cache_kernel_launches(self.handle))

    def corm_cache_export_state(self, layer, seq, kv_head, stream=None):
        """Live entries of one unit in slot order: k, v as float32 arrays [live, d], word, pos, counters."""
        c = self.cfg
        vt = _np_view_dtype(self.kv_dtype)
        k = np.empty((c.max_tokens, c.head_dim), dtype=vt)
        v = np.empty((c.max_tokens, c.head_dim), dtype=vt)
        word = np.empty((c.max_tokens,), dtype=np.uint32)
        pos = np.empty((c.max_tokens,), dtype=np.int32)
        live, n_tokens, n_obs = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check("corm_cache_export_state", self.lib.corm_cache_export_state(
            self.handle, layer, seq, kv_head, k.ctypes.data, v.ctypes.data, word.ctypes.data, pos.ctypes.data,
            ctypes.byref(live), ctypes.byref(n_tokens), ctypes.byref(n_obs), _stream_ptr(stream)))
        n = live.value
        widen = (lambda a: (a[:n].astype(np.uint32) << 16).view(np.float32)) if self.kv_dtype == CORM_BF16 else (
            lambda a: a[:n].copy())
        return dict(k=widen(k), v=widen(v), word=word[:n].copy(), pos=pos[:n].copy(), live_len=n,
                    n_tokens=n_tokens.value, n_obs=n_obs.value)

    def corm_cache_import_state(self, layer, seq, kv_head, k, v, word, pos, n_tokens, n_obs, stream=None):
        """k, v: float arrays [live, d] whose values are representable in the cache dtype."""
        k32 = np.ascontiguousarray(k, dtype=np.float32)
        v32 = np.ascontiguousarray(v, dtype=np.float32)
        if self.kv_dtype == CORM_BF16:
            assert not (k32.view(np.uint32) & 0xffff).any() and not (v32.view(np.uint32) & 0xffff).any()
            kk = np.ascontiguousarray((k32.view(np.uint32) >> 16).astype(np.uint16))
            vv = np.ascontiguousarray((v32.view(np.uint32) >> 16).astype(np.uint16))
        else:
            kk, vv = k32, v32
        word = np.ascontiguousarray(word, dtype=np.uint32)
        pos = np.ascontiguousarray(pos, dtype=np.int32)
        _check("corm_cache_import_state", self.lib.corm_cache_import_state(
            self.handle, layer, seq, kv_head, kk.ctypes.data, vv.ctypes.data, word.ctypes.data, pos.ctypes.data,
            int(kk.shape[0]), int(n_tokens), int(n_obs), _stream_ptr(stream)))
