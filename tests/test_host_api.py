"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the header declares, sizes its
arena as documented and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2404_15949_b200 import binding
from paper_2404_15949_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "corm.h")).read()
    names = set(re.findall(r"\b(corm_[a-z_]+)\s*\(", header))
    assert {"corm_cache_create", "corm_compress_prompt", "corm_decode_step", "corm_cache_stats"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} is declared in corm.h but not exported"


def _cfg(**kw):
    base = dict(n_layers=1, batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, max_tokens=512, window_w=8, recent_r=32,
                alpha=1.0, kv_dtype=binding.CORM_BF16, device=0)
    base.update(kw)
    return binding.CormConfig(*[base[k] for k, _ in binding.CormConfig._fields_])


def test_arena_bytes_and_the_256_gb_example(lib):
    # The introduction's example: a 7B model (32 layers x 32 heads x 128), batch 128, sequence 4096, 16-bit cache
    # needs 256 GB for K and V: 2 * 32*32*128 * 2 B = 0.5 MiB per token, times 4096 * 128 tokens = 256 GiB.
    kv = 2 * 32 * 32 * 128 * 2 * 4096 * 128
    assert kv == 256 * 2 ** 30
    total = binding.corm_cache_arena_bytes(_cfg(n_layers=32, batch=128, n_q_heads=32, n_kv_heads=32, max_tokens=4096))
    assert kv < total < kv * 1.03                                      # registers, positions and scratch: < 3 %
    assert binding.corm_cache_arena_bytes(_cfg(kv_dtype=binding.CORM_F32)) > binding.corm_cache_arena_bytes(_cfg())


@pytest.mark.parametrize("bad", [dict(n_q_heads=7), dict(recent_r=0), dict(window_w=0), dict(alpha=-1.0),
                                 dict(kv_dtype=5), dict(batch=0)])
def test_invalid_configs_have_no_arena(lib, bad):
    assert binding.corm_cache_arena_bytes(_cfg(**bad)) == 0


def test_create_rejects_before_any_cuda_call(lib):
    handle = ctypes.c_void_p()
    fake = ctypes.c_void_p(0x10000)                                    # aligned, never dereferenced on these paths
    cfg = _cfg()
    need = binding.corm_cache_arena_bytes(cfg)
    assert lib.corm_cache_create(ctypes.byref(cfg), fake, need - 1, ctypes.byref(handle)) == 3
    assert lib.corm_cache_create(ctypes.byref(cfg), None, need, ctypes.byref(handle)) == 1
    assert lib.corm_cache_create(ctypes.byref(cfg), ctypes.c_void_p(0x10001), need, ctypes.byref(handle)) == 1
    for bad, code in [(dict(head_dim=96), 2), (dict(window_w=257), 2), (dict(n_q_heads=6, n_kv_heads=2), 2),
                      (dict(n_q_heads=7), 1)]:
        c = _cfg(**bad)
        assert lib.corm_cache_create(ctypes.byref(c), fake, 1 << 40, ctypes.byref(handle)) == code
    assert handle.value is None
    assert lib.corm_status_string(6) == b"slab capacity exceeded"
    assert lib.corm_cache_destroy(None) == 1 and lib.corm_cache_kernel_launches(None) == 0


def test_step_calls_reject_a_missing_cache_before_any_cuda_call(lib):
    fake = ctypes.c_void_p(0x10000)
    assert lib.corm_decode_step(None, 0, fake, fake, fake, fake, None) == 1
    assert lib.corm_decode_step_layers(None, 0, 1, fake, fake, fake, fake, None) == 1
    assert lib.corm_decode_steps(None, 0, 1, 4, fake, fake, fake, fake, None) == 1
    assert lib.corm_decode_steps_host(None, 0, 1, 4, fake, fake, fake, fake, None) == 1
    assert lib.corm_decode_step_host(None, 0, fake, fake, fake, fake, None) == 1
    assert lib.corm_decode_step_static(None, 0, fake, fake, fake, fake, None) == 1
    assert lib.corm_cache_chained_launches(None) == 0
    assert len(lib.corm_status_string(8)) > 0 and lib.corm_status_string(8) != lib.corm_status_string(7)


def test_paged_arena_holds_the_pool_not_the_slabs(lib):
    # The paper's headline is up to 70 % of the KV cache saved: a pool sized for 30 % of the slabs' rows must need
    # about 30 % of the memory (page tables, bitmap, registers, positions and scratch on top).
    cfg = _cfg(n_layers=4, batch=8, n_q_heads=32, n_kv_heads=32, max_tokens=4096)
    slab = binding.corm_cache_arena_bytes(cfg)
    units, pages_per_slab = 8 * 32, 4096 // 32
    pool = units * pages_per_slab * 3 // 10 // 32 * 32
    paged = lib.corm_cache_arena_bytes_paged(ctypes.byref(cfg), pool)
    kv_pool = 4 * pool * 32 * 128 * 2 * 2
    assert kv_pool < paged < kv_pool + 0.07 * slab and paged < 0.37 * slab
    assert lib.corm_cache_arena_bytes_paged(ctypes.byref(cfg), 0) == slab            # 0 pages = slabs
    for bad in (units - 32, units + 1, -32):                                         # too few pages / not a multiple of 32
        assert lib.corm_cache_arena_bytes_paged(ctypes.byref(cfg), bad) == 0
    handle = ctypes.c_void_p()
    fake = ctypes.c_void_p(0x10000)
    assert lib.corm_cache_create_paged(ctypes.byref(cfg), units + 1, fake, 1 << 40, ctypes.byref(handle)) == 1
    assert lib.corm_cache_create_paged(ctypes.byref(cfg), pool, fake, paged - 1, ctypes.byref(handle)) == 3
    assert handle.value is None


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libcorm.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()
