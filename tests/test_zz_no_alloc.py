"""The allocation-free decode entry point (collected last on purpose).

``corm_decode_step_static`` is for callers that are handed a fixed set of device buffers and may not allocate where
the step runs (a plugin under a serving runtime with a frozen memory plan, an embedder without an allocator). It
keeps the step's scratch in an array built into the library, shared by every cache on the device, which still
holds the previous call's contents when the next call starts. The test therefore runs it twice in a row per cache,
interleaves two caches of different shapes on the same array, and requires the results of the ordinary entry
point: identical output bits (both run the same arithmetic) and identical cache state.
"""
import numpy as np
import pytest
import torch

from paper_2404_15949_b200.workload import CONFIGS, generate
from parity_util import OUT_TOL, make_gpu_cache, sorted_state, to_dev

pytestmark = pytest.mark.gpu


def _setup(cfg, fast):
    data = generate(cfg)
    nb, nh = len(data.seqs), len(data.kv_heads)
    ref, sta = make_gpu_cache(cfg, nb, nh), make_gpu_cache(cfg, nb, nh)
    dt = cfg.dtype
    for g in (ref, sta):
        g.corm_cache_set_tuning(0, fast)
        g.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                               data.prompt_lens)
    return data, ref, sta, nb, nh


def _step_and_compare(cfg, data, ref, sta, nb, nh, s):
    dt = cfg.dtype
    q, k, v = to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt)
    a = ref.corm_decode_step(0, q, k, v)
    out = torch.empty_like(q)
    b = sta.corm_decode_step_static(0, q, k, v, out)
    torch.cuda.synchronize()
    assert float((a.float() - b.float()).abs().max()) <= OUT_TOL[dt]
    for ib in range(nb):
        for ih in range(nh):
            x = sorted_state(ref.corm_cache_export_state(0, ib, ih))
            y = sorted_state(sta.corm_cache_export_state(0, ib, ih))
            assert x["live_len"] == y["live_len"]
            for key in ("pos", "word", "k", "v"):
                assert np.array_equal(x[key], y[key]), (s, ib, ih, key)


def test_static_scratch_entry_point_matches_on_consecutive_calls():
    cfg_a = CONFIGS[1].with_(prompt_min=300, prompt_max=300, steps=12)                       # fp32, 8 units
    cfg_b = CONFIGS[4].with_(batch=2, n_q_heads=8, n_kv_heads=2, prompt_min=500, prompt_max=700, steps=12,
                             recent_r=64, seed=4242)                                          # bf16, grouped queries
    A = _setup(cfg_a, False)
    B = _setup(cfg_b, False)
    for s in range(12):                    # consecutive calls; the two caches take turns on the shared array
        _step_and_compare(cfg_a, *A, s)
        _step_and_compare(cfg_b, *B, s)
    assert A[2].corm_cache_stats()["device_status"] == 0 and B[2].corm_cache_stats()["device_status"] == 0
    assert A[2].corm_cache_stats()["evicted_keys"] == A[1].corm_cache_stats()["evicted_keys"] > 0


def test_static_scratch_steps_against_the_oracle_without_allocating():
    """The entry point against the CPU oracle directly (outputs within tolerance, state bit-exact), and the property
    it exists for: with `out` supplied, a call makes no request to torch's allocator and takes no memory from the
    device (one warm-up call first: it looks up the built-in array's address and loads the kernel)."""
    from parity_util import assert_states_equal, make_oracle
    cfg = CONFIGS[4].with_(batch=2, n_q_heads=8, n_kv_heads=2, prompt_min=300, prompt_max=420, steps=16, recent_r=32,
                           seed=777)
    data = generate(cfg)
    nb, nh, dt = len(data.seqs), len(data.kv_heads), cfg.dtype
    gpu, orc = make_gpu_cache(cfg, nb, nh), make_oracle(cfg, nb, nh)
    gpu.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    orc.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    q, k, v = to_dev(data.q, dt), to_dev(data.k_new, dt), to_dev(data.v_new, dt)
    out = torch.empty_like(q[0])
    for s in range(cfg.steps):
        if s >= 1:
            torch.cuda.synchronize()
            n_allocs, free = torch.cuda.memory_stats()["allocation.all.allocated"], torch.cuda.mem_get_info()[0]
        gpu.corm_decode_step_static(0, q[s], k[s], v[s], out)
        if s >= 1:
            torch.cuda.synchronize()
            assert torch.cuda.memory_stats()["allocation.all.allocated"] == n_allocs, f"step {s}: torch allocated"
            assert torch.cuda.mem_get_info()[0] >= free, f"step {s}: device memory was taken"
        ref = orc.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
        assert np.abs(out.float().cpu().numpy() - ref).max() <= OUT_TOL[dt], f"step {s}"
        if s % 4 == 3 or s == cfg.steps - 1:
            assert_states_equal(gpu, orc, 0, nb, nh, f"after step {s}")
    assert orc.counters()["near_threshold"] == 0 and orc.counters()["evicted"] > 0
    assert gpu.corm_cache_stats()["device_status"] == 0


def test_static_scratch_rejects_oversized_caches():
    from paper_2404_15949_b200.binding import CormError
    cfg = CONFIGS[3].with_(batch=8, prompt_min=64, prompt_max=64, steps=4)                   # 256 units x 4608 slots
    data = generate(cfg.with_(prompt_min=64, prompt_max=64), n_steps=1)
    gpu = make_gpu_cache(cfg, 8, 32, max_tokens=16384)
    dt = cfg.dtype
    gpu.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    q, k, v = to_dev(data.q[0], dt), to_dev(data.k_new[0], dt), to_dev(data.v_new[0], dt)
    with pytest.raises(CormError) as e:
        gpu.corm_decode_step_static(0, q, k, v)                     # 256 * 16384 * 8 B of logits alone exceed 16 MiB
    assert e.value.status == 6
    assert (gpu.corm_cache_live_lens(0) == 64).all()                # nothing was enqueued
    gpu.corm_decode_step(0, q, k, v)                                # the arena path still works
    assert (gpu.corm_cache_live_lens(0) == 65).all()
