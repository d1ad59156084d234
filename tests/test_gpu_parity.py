"""GPU parity: the CUDA library against the CPU oracle through the C ABI, same seeded inputs on both sides.

Outputs must agree within max-abs 2e-3 (fp32 caches) / 2e-2 (bf16 caches); verdict registers, live-index lists and
cached rows must be bit-exact. The oracle's count of probabilities within 1e-6 (relative) of the threshold is
asserted to be zero on the fixed seeds, so no verdict is excused.
"""
import numpy as np
import pytest
import torch

from paper_2404_15949_b200.workload import CONFIGS, generate
from parity_util import (OUT_TOL, assert_states_equal, make_gpu_cache, make_oracle, run_free, sorted_state, to_dev)

pytestmark = pytest.mark.gpu


def _pair(cfg, data, **kw):
    nb, nh = len(data.seqs), len(data.kv_heads)
    return make_gpu_cache(cfg, nb, nh, **kw), make_oracle(cfg, nb, nh, **kw)


@pytest.mark.parametrize("split_len", [0, 64, 128])
def test_config1_tiny_f32_free_run(split_len):
    cfg = CONFIGS[1]
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    gpu.corm_cache_set_tuning(split_len, True)
    run_free(cfg, data, gpu, orc)
    c = orc.counters()
    assert c["near_threshold"] == 0 and c["evicted"] > 0
    st = gpu.corm_cache_stats()
    assert st["appended_keys"] == c["appended"] and st["evicted_keys"] == c["evicted"]
    assert st["live_keys"] == int(orc.live_lens(0).sum())


@pytest.mark.parametrize("seed", [15950, 15951])
def test_config1_other_seeds(seed):
    cfg = CONFIGS[1].with_(seed=seed)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    run_free(cfg, data, gpu, orc, check_every=8)
    assert orc.counters()["near_threshold"] == 0


SMALL = [
    # dtype, head_dim, group, n_kv, batch, prompt range, steps, w, r, split_len, fast
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 64, True),
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 64, 2),      # units of several splits finished inside the decode launch
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 64, 3),      # ... by the verdict launch
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 64, False),
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 128, True),     # grouped heads: the balanced kernel by default
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 128, 2),
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 128, 3),
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 0, 4),       # the balanced kernel forced for one head per KV head
    ("bf16", 128, 2, 2, 1, (31, 33), 70, 8, 32, 0, 4),
    ("bf16", 128, 4, 5, 3, (1, 40), 60, 8, 4, 0, 4),           # tiny units: many segments per block, units of one tile
    ("bf16", 128, 4, 1, 1, (3000, 3000), 12, 8, 64, 0, 4),     # one long unit cut over many blocks
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 0, 5),         # balanced streaming, verdicts by the verdict launch
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 0, 5),
    ("bf16", 128, 4, 5, 3, (1, 40), 60, 8, 4, 0, 5),
    ("bf16", 128, 4, 1, 1, (3000, 3000), 12, 8, 64, 0, 5),
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 128, False),
    ("bf16", 128, 8, 1, 2, (64, 129), 20, 3, 5, 64, True),
    ("bf16", 128, 2, 2, 1, (31, 33), 70, 8, 32, 64, True),
    ("bf16", 64, 4, 2, 2, (100, 200), 24, 8, 16, 64, True),
    ("f32", 64, 1, 2, 2, (60, 130), 24, 5, 7, 64, True),
    ("f32", 128, 8, 1, 1, (90, 90), 16, 16, 4, 0, True),
    ("f32", 128, 2, 2, 3, (0, 40), 40, 8, 3, 64, True),      # prompts shorter than w, including empty ones
]


@pytest.mark.parametrize("case", SMALL, ids=lambda c: "-".join(str(x) for x in c))
def test_small_shapes(case):
    dtype, d, G, nkv, B, (pmin, pmax), steps, w, r, split_len, fast = case
    cfg = CONFIGS[1].with_(name="small", batch=B, n_q_heads=nkv * G, n_kv_heads=nkv, head_dim=d, dtype=dtype,
                           prompt_min=pmin, prompt_max=pmax, steps=steps, window_w=w, recent_r=r,
                           gqa_rho=0.7 if G > 1 else 0.0, hh_min=2, hh_max=6, seed=777)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    gpu.corm_cache_set_tuning(split_len, fast)
    run_free(cfg, data, gpu, orc)
    assert orc.counters()["near_threshold"] == 0


@pytest.mark.parametrize("dtype,d,G", [("bf16", 128, 1), ("bf16", 128, 4), ("f32", 64, 2)])
def test_adjacent_query_similarity_monitor(dtype, d, G):
    """Eq. 3 between consecutive decode queries, summed by the opt-in monitor, against the oracle's fp64 sum."""
    cfg = CONFIGS[1].with_(name="sim", batch=2, n_q_heads=2 * G, n_kv_heads=2, head_dim=d, dtype=dtype, prompt_min=90,
                           prompt_max=160, steps=20, gqa_rho=0.7 if G > 1 else 0.0, seed=321)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    gpu.corm_cache_set_similarity_monitor(True)
    run_free(cfg, data, gpu, orc, check_every=10)
    (sg, ng), (so, no) = gpu.corm_cache_similarity(), orc.similarity()
    assert ng == no == 2 * 2 * G * (cfg.steps - 1)
    assert abs(sg - so) <= 1e-9 * no
    assert 0.0 < so / no < 1.0                                   # the generator's queries drift slowly (Section 3.3)


@pytest.mark.parametrize("G,w,scale", [(1, 8, 1.0), (4, 8, 1e3), (1, 8, 1e12), (4, 40, 1e12)])
def test_prompt_pass_fp32_placement_and_exact_path(G, w, scale):
    """Second launch of the tiled prompt pass: fp32 logits against exact thresholds where a proven error bound allows,
    fp64 again where it does not. Inflating the bound (at 1e12: every logit) must not change a single register."""
    cfg = CONFIGS[1].with_(name="prompt32", batch=2, n_q_heads=2 * G, n_kv_heads=2, head_dim=128, dtype="bf16",
                           prompt_min=500, prompt_max=900, steps=4, window_w=w, recent_r=16,
                           gqa_rho=0.7 if G > 1 else 0.0, hh_min=2, hh_max=6, seed=578)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    gpu.corm_cache_set_bound_scale(scale)
    run_free(cfg, data, gpu, orc)
    assert orc.counters()["near_threshold"] == 0 and orc.counters()["evicted"] > 0


def test_alpha_zero_never_evicts():
    cfg = CONFIGS[1].with_(prompt_min=100, prompt_max=100, steps=20, alpha=0.0, dtype="bf16")
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    run_free(cfg, data, gpu, orc)
    assert (gpu.corm_cache_live_lens(0) == 120).all()
    assert gpu.corm_cache_stats()["evicted_keys"] == 0


def test_lockstep_from_imported_state():
    """Both sides start every step from the oracle's state (import hook), as the large configurations do."""
    cfg = CONFIGS[1].with_(prompt_min=200, prompt_max=200, steps=24, dtype="bf16", n_q_heads=8, n_kv_heads=2,
                           gqa_rho=0.7)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    orc.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    dt = cfg.dtype
    for s in range(cfg.steps):
        for h in range(2):
            st = orc.export_unit(0, 0, h)
            perm = np.random.default_rng(s * 7 + h).permutation(st["live_len"])      # slot order is free
            gpu.corm_cache_import_state(0, 0, h, st["k"][perm], st["v"][perm], st["word"][perm], st["pos"][perm],
                                        st["n_tokens"], st["n_obs"])
        out_g = gpu.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
        out_o = orc.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
        assert np.abs(out_g.float().cpu().numpy() - out_o).max() <= OUT_TOL[dt]
        assert_states_equal(gpu, orc, 0, 1, 2, f"step {s}")


def test_multi_layer_independent_and_deterministic():
    cfg = CONFIGS[2].with_(n_layers=3, n_q_heads=4, n_kv_heads=4, prompt_min=300, prompt_max=300, steps=12,
                           recent_r=32, dense_layers=1)
    gpu = make_gpu_cache(cfg, 1, 4, n_layers=3)
    gpu2 = make_gpu_cache(cfg, 1, 4, n_layers=3)
    orc = make_oracle(cfg, 1, 4, n_layers=3)
    datas = [generate(cfg, layer=l) for l in range(3)]
    dt = cfg.dtype
    for l in (2, 0, 1):                                              # layers in any order
        d = datas[l]
        for g in (gpu, gpu2):
            g.corm_compress_prompt(l, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
        orc.compress_prompt(l, d.k_prompt, d.v_prompt, d.q_last, d.prompt_lens)
    for s in range(cfg.steps):
        for l in (1, 2, 0):
            d = datas[l]
            a = gpu.corm_decode_step(l, to_dev(d.q[s], dt), to_dev(d.k_new[s], dt), to_dev(d.v_new[s], dt))
            b = gpu2.corm_decode_step(l, to_dev(d.q[s], dt), to_dev(d.k_new[s], dt), to_dev(d.v_new[s], dt))
            o = orc.decode_step(l, d.q[s], d.k_new[s], d.v_new[s])
            assert torch.equal(a, b)                                  # same inputs twice -> identical bits
            assert np.abs(a.float().cpu().numpy() - o).max() <= OUT_TOL[dt]
    for l in range(3):
        assert_states_equal(gpu, orc, l, 1, 4, f"layer {l}")
        for h in range(4):
            sa = sorted_state(gpu.corm_cache_export_state(l, 0, h))
            sb = sorted_state(gpu2.corm_cache_export_state(l, 0, h))
            assert all(np.array_equal(sa[k], sb[k]) for k in ("k", "v", "word", "pos"))
    # two launches per prompt pass; per step one streaming launch, plus a verdict launch while units span several splits
    n = gpu.corm_cache_kernel_launches()
    assert 2 * 3 + 3 * cfg.steps <= n <= 2 * 3 + 2 * 3 * cfg.steps and n == gpu2.corm_cache_kernel_launches()


@pytest.mark.parametrize("G", [1, 4])
def test_all_layers_from_one_call_equal_per_layer_calls(G):
    """corm_decode_step_layers is n per-layer calls in layer order. With separate tensors per layer it enqueues those
    calls (identical output bits); with the layers' tensors contiguous it steps all layers by ONE launch (pair), whose
    blocks are cut differently, so outputs agree within rounding. Either way the states equal the oracle's."""
    from paper_2404_15949_b200.binding import CormError
    cfg = CONFIGS[2].with_(n_layers=4, n_q_heads=4 * G, n_kv_heads=4, prompt_min=260, prompt_max=260, steps=14,
                           recent_r=32, dense_layers=1, gqa_rho=0.7 if G > 1 else 0.0)
    one, many = make_gpu_cache(cfg, 1, 4, n_layers=4), make_gpu_cache(cfg, 1, 4, n_layers=4)
    orc = make_oracle(cfg, 1, 4, n_layers=4)
    datas = [generate(cfg, layer=l) for l in range(4)]
    dt = cfg.dtype
    for l, d in enumerate(datas):
        for g in (one, many):
            g.corm_compress_prompt(l, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
        orc.compress_prompt(l, d.k_prompt, d.v_prompt, d.q_last, d.prompt_lens)
    launches_fused = 0
    for s in range(cfg.steps):
        q_all = torch.stack([to_dev(d.q[s], dt) for d in datas]).contiguous()
        k_all = torch.stack([to_dev(d.k_new[s], dt) for d in datas]).contiguous()
        v_all = torch.stack([to_dev(d.v_new[s], dt) for d in datas]).contiguous()
        fused = s % 3 != 2                                             # two steps by one launch, then one step layer by layer
        if fused:
            q, k, v = list(q_all), list(k_all), list(v_all)
            out_all = torch.empty_like(q_all)
            outs = list(out_all)
        else:
            q, k, v = [x.clone() for x in q_all], [x.clone() for x in k_all], [x.clone() for x in v_all]
            outs = [torch.empty_like(x) for x in q]
        before = many.corm_cache_kernel_launches()
        if s % 2:
            many.corm_decode_step_layers(0, q, k, v, outs)
        else:
            many.corm_decode_step_layers(0, many.pointer_table(q, "q"), many.pointer_table(k, "kv"),
                                         many.pointer_table(v, "kv"), many.pointer_table(outs, "q"))
        n_l = many.corm_cache_kernel_launches() - before
        assert n_l <= 2 if fused else n_l >= 4, (s, n_l)
        launches_fused += fused
        for l in range(4):
            a = one.corm_decode_step(l, q[l], k[l], v[l])
            ref = orc.decode_step(l, datas[l].q[s], datas[l].k_new[s], datas[l].v_new[s])
            if fused:
                assert np.abs(outs[l].float().cpu().numpy() - ref).max() <= OUT_TOL[dt]
            else:
                assert torch.equal(a, outs[l])
            assert np.abs(a.float().cpu().numpy() - ref).max() <= OUT_TOL[dt]
        if s % 4 == 3:
            for l in range(4):
                assert_states_equal(many, orc, l, 1, 4, f"step {s} layer {l}")
    for l in range(4):
        assert_states_equal(many, orc, l, 1, 4, f"layer {l}")
        assert_states_equal(one, orc, l, 1, 4, f"layer {l}")
    assert many.corm_cache_stats()["evicted_keys"] == one.corm_cache_stats()["evicted_keys"] == orc.counters()["evicted"] > 0
    before = many.corm_cache_kernel_launches()
    with pytest.raises(CormError):
        many.corm_decode_step_layers(2, q, k, v, outs)                 # layers 2..5 of 4
    assert many.corm_cache_kernel_launches() == before


WIDE = [
    # dtype, d, G, n_kv, B, prompt range, steps, w, r, split_len, fast, alpha, seed
    ("bf16", 128, 1, 4, 2, (300, 520), 80, 40, 16, 0, True, 1.0, 4242),      # tiled prompt pass, one launch pair
    ("bf16", 128, 1, 2, 2, (20, 90), 150, 64, 8, 0, True, 1.0, 4245),        # prompts near the window size; it fills in decode
    ("bf16", 128, 4, 2, 2, (400, 900), 60, 48, 32, 128, True, 2.0, 4242),    # GQA, three launch pairs, multi-split decode
    ("bf16", 128, 1, 2, 1, (1500, 1500), 40, 256, 256, 0, True, 6.0, 4242),  # the paper's 256 + 256 budget
    ("bf16", 128, 4, 1, 1, (700, 700), 300, 256, 64, 0, True, 6.0, 4243),    # 256-query window, 16 launch pairs
    ("f32", 64, 2, 2, 2, (150, 260), 70, 100, 10, 64, False, 1.5, 4242),     # generic kernels, chunked prompt rows
    ("bf16", 128, 8, 1, 1, (300, 300), 50, 33, 4, 0, True, 1.0, 4243),       # group of 8: generic decode, tiled prompt
]


@pytest.mark.parametrize("case", WIDE, ids=lambda c: "-".join(str(x) for x in c))
def test_windows_beyond_32_queries(case):
    """Windows of 33..256 queries keep, per key, the step of its latest important verdict instead of a shift register;
    live lists, rows and the visible part of every register must still match the oracle's multi-word registers."""
    dtype, d, G, nkv, B, (pmin, pmax), steps, w, r, split_len, fast, alpha, seed = case
    cfg = CONFIGS[1].with_(name="wide", batch=B, n_q_heads=nkv * G, n_kv_heads=nkv, head_dim=d, dtype=dtype,
                           prompt_min=pmin, prompt_max=pmax, steps=steps, window_w=w, recent_r=r, alpha=alpha,
                           gqa_rho=0.7 if G > 1 else 0.0, hh_min=2, hh_max=6, seed=seed)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    gpu.corm_cache_set_tuning(split_len, fast)
    run_free(cfg, data, gpu, orc, check_every=5)
    assert orc.counters()["near_threshold"] == 0
    assert gpu.corm_cache_stats()["evicted_keys"] > 0


def test_wide_window_import_roundtrip():
    """Importing the oracle's state (ages turned into stamps) and stepping gives the oracle's next state."""
    from parity_util import ages_to_stamps
    cfg = CONFIGS[1].with_(prompt_min=260, prompt_max=260, steps=30, dtype="bf16", n_q_heads=2, n_kv_heads=2,
                           window_w=70, recent_r=12)
    data = generate(cfg)
    gpu, orc = _pair(cfg, data)
    orc.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    dt = cfg.dtype
    for s in range(cfg.steps):
        for h in range(2):
            st = orc.export_unit(0, 0, h)
            gpu.corm_cache_import_state(0, 0, h, st["k"], st["v"], ages_to_stamps(st["age"], st["n_tokens"]),
                                        st["pos"], st["n_tokens"], st["n_obs"])
        out_g = gpu.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
        out_o = orc.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
        assert np.abs(out_g.float().cpu().numpy() - out_o).max() <= OUT_TOL[dt]
        assert_states_equal(gpu, orc, 0, 1, 2, f"step {s}")


@pytest.mark.parametrize("pinned", [True, False], ids=["pinned-in-place", "pageable-staged"])
def test_host_buffer_entry_point_matches_device_one(pinned):
    """Pinned buffers are read and written by the kernels in place; pageable ones go through the arena's staging
    space. Either way the step equals the device-buffer call bit for bit."""
    cfg = CONFIGS[1].with_(prompt_min=130, prompt_max=130, steps=10, dtype="bf16")
    data = generate(cfg)
    a, b = make_gpu_cache(cfg, 1, 8), make_gpu_cache(cfg, 1, 8)
    dt = cfg.dtype
    for g in (a, b):
        g.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                               data.prompt_lens)

    def host(x):
        t = torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)
        return t.pin_memory() if pinned else t

    for s in range(cfg.steps):
        ref = a.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
        out = host(np.zeros(tuple(ref.shape), dtype=np.float32))
        b.corm_decode_step_host(0, host(data.q[s]), host(data.k_new[s]), host(data.v_new[s]), out)
        torch.cuda.synchronize()
        assert torch.equal(ref.cpu(), out)
    for h in range(8):
        sa, sb = sorted_state(a.corm_cache_export_state(0, 0, h)), sorted_state(b.corm_cache_export_state(0, 0, h))
        assert all(np.array_equal(sa[k], sb[k]) for k in ("k", "v", "word", "pos"))


def test_capacity_overflow_is_reported_not_fatal():
    cfg = CONFIGS[1].with_(prompt_min=40, prompt_max=40, steps=8, alpha=0.0, n_q_heads=2, n_kv_heads=2)
    data = generate(cfg)
    gpu = make_gpu_cache(cfg, 1, 2, max_tokens=44)
    dt = cfg.dtype
    gpu.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    for s in range(6):
        gpu.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
    st = gpu.corm_cache_stats()
    assert st["device_status"] == 6 and (gpu.corm_cache_live_lens(0) == 44).all()


def test_state_errors_on_gpu():
    from paper_2404_15949_b200.binding import CormError
    cfg = CONFIGS[1].with_(n_q_heads=2, n_kv_heads=2)
    gpu = make_gpu_cache(cfg, 1, 2)
    x = torch.zeros(1, 2, 128, device="cuda")
    with pytest.raises(CormError) as e:
        gpu.corm_decode_step(0, x, x, x)                             # no prompt pass yet
    assert e.value.status == 4
    with pytest.raises(CormError):
        gpu.corm_decode_step(1, x, x, x)                             # layer out of range


CHAINED = [
    # G, n_kv, batch, layers, prompt range, steps, w, r, split_len, tuning, pool_pages
    (1, 32, 10, 1, (150, 500), 44, 8, 32, 0, 1, 0),        # 320 short units: one block each, every launch self-finishing
    (1, 32, 10, 1, (150, 500), 44, 8, 32, 0, 1, 8192),     # ... on a paged cache
    (1, 3, 2, 1, (150, 330), 40, 8, 16, 64, 2, 0),         # units of several splits, finished by the last-arriving split
    (4, 2, 2, 1, (97, 257), 36, 4, 8, 128, 2, 0),          # grouped heads on the block-per-split kernel
    (1, 8, 1, 4, (260, 260), 30, 8, 32, 0, 1, 0),          # four layers as one launch per step
    (4, 2, 2, 1, (97, 257), 36, 4, 8, 0, 1, 0),            # grouped heads, automatic: a block per split inside such a call
    (4, 1, 1, 1, (3000, 3000), 12, 8, 64, 0, 1, 0),        # one long unit: balanced kernel + verdict launch, nothing to chain
    (4, 8, 6, 1, (150, 700), 44, 8, 32, 128, 6, 0),        # grouped heads, tensor-core loop, a block per split of 128 keys
    (4, 8, 6, 1, (150, 700), 44, 8, 32, 0, 6, 4096),       # ... automatic split length, paged cache
    (2, 3, 2, 1, (1, 40), 60, 8, 4, 0, 6, 0),              # tiny units (empty splits), two heads per group
    (1, 3, 2, 1, (150, 330), 40, 8, 16, 128, 6, 0),        # one head per KV head on that kernel
    (4, 2, 1, 3, (260, 260), 30, 8, 32, 0, 6, 0),          # three layers as one launch per step
    (1, 8, 1, 2, (260, 260), 20, 8, 32, 0, 1, 2048),       # two layers with pools of their own: a launch per layer, unchained
]


@pytest.mark.parametrize("G,n_kv,batch,n_layers,prange,steps,w,r,split_len,tuning,pool_pages", CHAINED)
def test_many_steps_from_one_call(G, n_kv, batch, n_layers, prange, steps, w, r, split_len, tuning, pool_pages):
    """corm_decode_steps: several decode steps enqueued by one call, each launch chained to the previous one where
    the kernels allow it (a block waits for its own unit's previous step only). Outputs of every step and the states
    between calls equal the oracle's, which steps one call at a time."""
    cfg = CONFIGS[2].with_(n_layers=n_layers, batch=batch, n_q_heads=n_kv * G, n_kv_heads=n_kv, prompt_min=prange[0],
                           prompt_max=prange[1], steps=steps, window_w=w, recent_r=r, dense_layers=0,
                           gqa_rho=0.7 if G > 1 else 0.0)
    gpu = make_gpu_cache(cfg, batch, n_kv, n_layers=n_layers, pool_pages=pool_pages)
    orc = make_oracle(cfg, batch, n_kv, n_layers=n_layers)
    gpu.corm_cache_set_tuning(split_len, tuning)
    datas = [generate(cfg, layer=l) for l in range(n_layers)]
    dt = cfg.dtype
    for l, d in enumerate(datas):
        gpu.corm_compress_prompt(l, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
        orc.compress_prompt(l, d.k_prompt, d.v_prompt, d.q_last, d.prompt_lens)
    q_all = torch.stack([to_dev(d.q[:steps], dt) for d in datas], dim=1).contiguous()      # [steps, layers, ...]
    k_all = torch.stack([to_dev(d.k_new[:steps], dt) for d in datas], dim=1).contiguous()
    v_all = torch.stack([to_dev(d.v_new[:steps], dt) for d in datas], dim=1).contiguous()
    s0 = 0
    for chunk in (1, 7, 16, 3, steps):                       # calls of different lengths, the last takes what is left
        s1 = min(steps, s0 + chunk)
        out = gpu.corm_decode_steps(0, n_layers, q_all[s0:s1], k_all[s0:s1], v_all[s0:s1]).float().cpu().numpy()
        for s in range(s0, s1):
            for l, d in enumerate(datas):
                ref = orc.decode_step(l, d.q[s], d.k_new[s], d.v_new[s])
                assert np.abs(out[s - s0, l] - ref).max() <= OUT_TOL[dt], (s, l)
        for l in range(n_layers):
            assert_states_equal(gpu, orc, l, batch, n_kv, f"after step {s1 - 1} layer {l}")
        s0 = s1
    st = gpu.corm_cache_stats()
    assert st["device_status"] == 0 and st["evicted_keys"] == orc.counters()["evicted"] > 0
    assert orc.counters()["near_threshold"] == 0
    chained = gpu.corm_cache_chained_launches()
    if (G > 1 and tuning == 1 and prange[1] > 96 * batch * n_kv * n_layers) or (pool_pages and n_layers > 1):
        assert chained == 0
    else:     # every launch after a call's first, as long as each finished its units itself
        assert chained >= steps // 2, chained
    if pool_pages:
        used, _ = gpu.corm_cache_pool_usage(0)
        assert used == int((orc.live_lens(0) // 32 + 1).sum())


@pytest.mark.parametrize("pinned", [True, False])
def test_many_steps_from_host_buffers(pinned):
    """corm_decode_steps_host: pinned buffers are read and written in place by the (chained) launches, pageable ones
    go through the staging buffers step by step; same results either way."""
    G, n_kv, batch, steps = 1, 32, 10, 24
    cfg = CONFIGS[2].with_(n_layers=1, batch=batch, n_q_heads=n_kv * G, n_kv_heads=n_kv, prompt_min=150, prompt_max=400,
                           steps=steps, window_w=8, recent_r=32, dense_layers=0)
    gpu, orc = make_gpu_cache(cfg, batch, n_kv), make_oracle(cfg, batch, n_kv)
    d = generate(cfg)
    dt = cfg.dtype
    gpu.corm_compress_prompt(0, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
    orc.compress_prompt(0, d.k_prompt, d.v_prompt, d.q_last, d.prompt_lens)
    host = lambda a: (lambda t: t.pin_memory() if pinned else t)(to_dev(a[:steps], dt).unsqueeze(1).contiguous().cpu())
    q, k, v = host(d.q), host(d.k_new), host(d.v_new)
    out = torch.empty_like(q)
    out = out.pin_memory() if pinned else out
    gpu.corm_decode_steps_host(0, 1, q, k, v, out)
    torch.cuda.synchronize()
    res = out.float().numpy()
    for s in range(steps):
        ref = orc.decode_step(0, d.q[s], d.k_new[s], d.v_new[s])
        assert np.abs(res[s, 0] - ref).max() <= OUT_TOL[dt], s
    assert_states_equal(gpu, orc, 0, batch, n_kv, "after the call")
    assert gpu.corm_cache_stats()["device_status"] == 0
    assert (gpu.corm_cache_chained_launches() > 0) == pinned
