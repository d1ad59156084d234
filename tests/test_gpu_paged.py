"""GPU parity of the paged cache (K and V in a pool of 32-key pages shared by a layer's units) against the CPU
oracle: same tolerances and bit-exact state as the slab cache, plus the pool's own invariants. Between steps a unit
of n live keys holds n // 32 + 1 pages, so the pages in use must equal the sum of that over the units, every step,
whichever kernel finished the unit (on-chip finish, last-arriving split, verdict launch, generic kernel)."""
import numpy as np
import pytest

from paper_2404_15949_b200.workload import CONFIGS, generate
from parity_util import OUT_TOL, assert_states_equal, make_gpu_cache, make_oracle, to_dev

pytestmark = pytest.mark.gpu


def _pages_expected(live):
    return int((np.asarray(live) // 32 + 1).sum())


PAGED = [
    # dtype, head_dim, group, n_kv, batch, prompt range, steps, w, r, split_len, fast, pool_pages
    ("bf16", 128, 1, 3, 2, (150, 330), 72, 8, 16, 0, True, 96),       # on-chip finish of single-split units
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 128, 2, 96),        # last-arriving split finishes the unit
    ("bf16", 128, 1, 3, 2, (150, 330), 40, 8, 16, 128, 3, 96),        # verdict launch
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 128, True, 64),       # balanced kernel (default for grouped heads)
    ("bf16", 128, 1, 3, 2, (150, 330), 72, 8, 16, 0, 4, 96),          # balanced kernel, one head per KV head
    ("bf16", 128, 4, 1, 1, (3000, 3000), 12, 8, 64, 0, 4, 128),       # one long unit cut over many blocks
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 0, 5, 64),            # balanced streaming + verdict launch
    ("bf16", 128, 4, 1, 1, (3000, 3000), 12, 8, 64, 0, 5, 128),
    ("bf16", 128, 4, 2, 2, (97, 257), 36, 4, 8, 128, 3, 64),
    ("bf16", 128, 2, 2, 1, (31, 33), 70, 8, 32, 0, True, 32),         # grows across page boundaries from one page
    ("bf16", 128, 8, 1, 2, (64, 129), 20, 3, 5, 64, True, 32),        # generic decode kernel, tiled prompt pass
    ("bf16", 64, 4, 2, 2, (100, 200), 24, 8, 16, 64, True, 64),       # generic kernels throughout
    ("f32", 128, 2, 2, 3, (0, 40), 40, 8, 3, 64, True, 32),           # empty and short prompts
    ("f32", 64, 1, 2, 2, (60, 130), 24, 5, 7, 64, True, 32),
]


@pytest.mark.parametrize("case", PAGED, ids=lambda c: "-".join(str(x) for x in c))
def test_paged_cache_matches_oracle_and_pool_accounting(case):
    dtype, d, G, nkv, B, (pmin, pmax), steps, w, r, split_len, fast, pool = case
    cfg = CONFIGS[1].with_(name="paged", batch=B, n_q_heads=nkv * G, n_kv_heads=nkv, head_dim=d, dtype=dtype,
                           prompt_min=pmin, prompt_max=pmax, steps=steps, window_w=w, recent_r=r,
                           gqa_rho=0.7 if G > 1 else 0.0, hh_min=2, hh_max=6, seed=777)
    data = generate(cfg)
    nb, nh = len(data.seqs), len(data.kv_heads)
    gpu, orc = make_gpu_cache(cfg, nb, nh, pool_pages=pool), make_oracle(cfg, nb, nh)
    gpu.corm_cache_set_tuning(split_len, fast)
    dt = cfg.dtype
    gpu.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    orc.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    assert_states_equal(gpu, orc, 0, nb, nh, "after prompt")
    assert gpu.corm_cache_pool_usage(0) == (_pages_expected(orc.live_lens(0)), pool)
    for s in range(steps):
        out_g = gpu.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
        out_o = orc.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
        assert np.abs(out_g.float().cpu().numpy() - out_o).max() <= OUT_TOL[dt], f"step {s}"
        assert gpu.corm_cache_pool_usage(0)[0] == _pages_expected(orc.live_lens(0)), f"pages in use after step {s}"
        if s % 4 == 3 or s == steps - 1:
            assert_states_equal(gpu, orc, 0, nb, nh, f"after step {s}")
    st = gpu.corm_cache_stats()
    assert st["device_status"] == 0 and orc.counters()["near_threshold"] == 0
    assert (st["important_keys"], st["attended_keys"]) == orc.sparsity()
    # a new prompt pass on the layer returns every page first
    gpu.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    assert gpu.corm_cache_pool_usage(0)[0] == _pages_expected(gpu.corm_cache_live_lens(0))


def test_paged_cache_equals_slab_cache_bit_for_bit():
    """Same inputs through a slab cache and a paged one: outputs, slot order, registers and rows are identical."""
    cfg = CONFIGS[1].with_(name="paged", batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype="bf16", prompt_min=700,
                           prompt_max=900, steps=48, window_w=8, recent_r=32, gqa_rho=0.7, seed=4242)
    data = generate(cfg)
    nb, nh = len(data.seqs), len(data.kv_heads)
    slab, paged = make_gpu_cache(cfg, nb, nh), make_gpu_cache(cfg, nb, nh, pool_pages=160)
    dt = cfg.dtype
    args = (to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt), data.prompt_lens)
    slab.corm_compress_prompt(0, *args)
    paged.corm_compress_prompt(0, *args)
    for s in range(cfg.steps):
        step = (to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
        a, b = slab.corm_decode_step(0, *step), paged.corm_decode_step(0, *step)
        assert (a == b).all(), f"step {s}"
    for b in range(nb):
        for h in range(nh):
            x, y = slab.corm_cache_export_state(0, b, h), paged.corm_cache_export_state(0, b, h)
            n = x["live_len"]
            assert n == y["live_len"] and x["n_tokens"] == y["n_tokens"]
            for key in ("k", "v", "word", "pos"):
                assert np.array_equal(x[key][:n], y[key][:n]), (b, h, key)
    used, total = paged.corm_cache_pool_usage(0)
    assert used == _pages_expected(paged.corm_cache_live_lens(0)) and total == 160
    assert paged.corm_cache_stats()["device_status"] == 0


def test_tight_pool_under_churn_equals_slab_cache():
    """256 units claim and release pages concurrently in a pool only a little larger than what they hold at the peak,
    so home regions overflow into their neighbours' and claims fall back to scanning the bitmap. Outputs must still
    equal the slab cache's bit for bit at every step, no page may be lost or held twice (pages in use = what the live
    lengths require, every 8 steps), and the final states must be identical."""
    cfg = CONFIGS[1].with_(name="churn", batch=8, n_q_heads=32, n_kv_heads=32, head_dim=128, dtype="bf16",
                           prompt_min=200, prompt_max=700, steps=160, window_w=4, recent_r=16, hh_min=2, hh_max=6,
                           seed=99)
    data = generate(cfg)
    nb, nh = len(data.seqs), len(data.kv_heads)
    dt = cfg.dtype
    slab = make_gpu_cache(cfg, nb, nh)
    args = (to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt), data.prompt_lens)
    slab.corm_compress_prompt(0, *args)
    need = _pages_expected(slab.corm_cache_live_lens(0))            # the peak: lengths only shrink towards r + a few
    pool = (need + 256 + 31) // 32 * 32                             # one spare page per unit
    paged = make_gpu_cache(cfg, nb, nh, pool_pages=pool)
    paged.corm_compress_prompt(0, *args)
    assert paged.corm_cache_pool_usage(0) == (need, pool)
    q, k, v = to_dev(data.q, dt), to_dev(data.k_new, dt), to_dev(data.v_new, dt)
    for s in range(cfg.steps):
        a, b = slab.corm_decode_step(0, q[s], k[s], v[s]), paged.corm_decode_step(0, q[s], k[s], v[s])
        assert (a == b).all(), f"step {s}"
        if s % 8 == 7:
            live = paged.corm_cache_live_lens(0)
            assert (live == slab.corm_cache_live_lens(0)).all()
            assert paged.corm_cache_pool_usage(0)[0] == _pages_expected(live), f"step {s}"
    assert paged.corm_cache_stats()["device_status"] == 0 and paged.corm_cache_stats()["evicted_keys"] > 0
    for b in range(0, nb, 3):
        for h in range(0, nh, 5):
            x, y = slab.corm_cache_export_state(0, b, h), paged.corm_cache_export_state(0, b, h)
            assert x["live_len"] == y["live_len"]
            assert all(np.array_equal(x[key], y[key]) for key in ("k", "v", "word", "pos")), (b, h)


def test_paged_lockstep_from_imported_state():
    """Import hook on a paged cache: the host hands the unit its pages; every step restarts from the oracle's state."""
    cfg = CONFIGS[1].with_(prompt_min=200, prompt_max=200, steps=12, dtype="bf16", n_q_heads=8, n_kv_heads=2,
                           gqa_rho=0.7)
    data = generate(cfg)
    gpu, orc = make_gpu_cache(cfg, 1, 2, pool_pages=32), make_oracle(cfg, 1, 2)
    orc.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    dt = cfg.dtype
    for s in range(cfg.steps):
        for h in range(2):
            st = orc.export_unit(0, 0, h)
            perm = np.random.default_rng(s * 7 + h).permutation(st["live_len"])
            gpu.corm_cache_import_state(0, 0, h, st["k"][perm], st["v"][perm], st["word"][perm], st["pos"][perm],
                                        st["n_tokens"], st["n_obs"])
        assert gpu.corm_cache_pool_usage(0)[0] == _pages_expected(orc.live_lens(0))
        out_g = gpu.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
        out_o = orc.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
        assert np.abs(out_g.float().cpu().numpy() - out_o).max() <= OUT_TOL[dt]
        assert_states_equal(gpu, orc, 0, 1, 2, f"step {s}")


@pytest.mark.parametrize("case", [
    ("bf16", 128, 4, 2, 2, (400, 900), 40, 48, 32, 128, True, 2.0, 4242, 128),   # stamps, three prompt launch pairs
    ("f32", 64, 2, 2, 2, (150, 260), 40, 100, 10, 64, False, 1.5, 4242, 64),     # generic kernels, chunked prompt rows
], ids=lambda c: "-".join(str(x) for x in c))
def test_paged_cache_with_windows_beyond_32_queries(case):
    from parity_util import run_free
    dtype, d, G, nkv, B, (pmin, pmax), steps, w, r, split_len, fast, alpha, seed, pool = case
    cfg = CONFIGS[1].with_(name="wide", batch=B, n_q_heads=nkv * G, n_kv_heads=nkv, head_dim=d, dtype=dtype,
                           prompt_min=pmin, prompt_max=pmax, steps=steps, window_w=w, recent_r=r, alpha=alpha,
                           gqa_rho=0.7 if G > 1 else 0.0, hh_min=2, hh_max=6, seed=seed)
    data = generate(cfg)
    nb, nh = len(data.seqs), len(data.kv_heads)
    gpu, orc = make_gpu_cache(cfg, nb, nh, pool_pages=pool), make_oracle(cfg, nb, nh)
    gpu.corm_cache_set_tuning(split_len, fast)
    run_free(cfg, data, gpu, orc, check_every=5)
    assert orc.counters()["near_threshold"] == 0 and gpu.corm_cache_stats()["evicted_keys"] > 0
    assert gpu.corm_cache_pool_usage(0)[0] == _pages_expected(orc.live_lens(0))


def test_paged_cache_through_the_host_buffer_and_static_scratch_entry_points():
    """The other two decode entry points on a paged cache: pinned host buffers read in place, and the step whose
    scratch lives inside the library. Each must leave the state the plain call leaves on a slab cache."""
    import torch
    cfg = CONFIGS[4].with_(batch=2, n_q_heads=8, n_kv_heads=2, prompt_min=500, prompt_max=700, steps=10,
                           recent_r=64, seed=4242)
    data = generate(cfg)
    nb, nh = len(data.seqs), len(data.kv_heads)
    dt = cfg.dtype
    ref = make_gpu_cache(cfg, nb, nh)
    hst, sta = make_gpu_cache(cfg, nb, nh, pool_pages=128), make_gpu_cache(cfg, nb, nh, pool_pages=128)
    for g in (ref, hst, sta):
        g.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                               data.prompt_lens)
    pin = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).pin_memory()
    for s in range(cfg.steps):
        q, k, v = to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt)
        a = ref.corm_decode_step(0, q, k, v)
        out_h = pin(np.zeros(tuple(a.shape), dtype=np.float32))
        hst.corm_decode_step_host(0, pin(data.q[s]), pin(data.k_new[s]), pin(data.v_new[s]), out_h)
        out_s = torch.empty_like(q)
        sta.corm_decode_step_static(0, q, k, v, out_s)
        torch.cuda.synchronize()
        assert torch.equal(a.cpu(), out_h)
        assert float((a.float() - out_s.float()).abs().max()) <= OUT_TOL[dt]
    for b in range(nb):
        for h in range(nh):
            x = ref.corm_cache_export_state(0, b, h)
            n = x["live_len"]
            y = hst.corm_cache_export_state(0, b, h)
            assert y["live_len"] == n and all(np.array_equal(x[key][:n], y[key][:n]) for key in ("k", "v", "word", "pos"))
            z = sta.corm_cache_export_state(0, b, h)      # the generic kernel may order slots differently: compare by position
            assert z["live_len"] == n
            ox, oz = np.argsort(x["pos"][:n]), np.argsort(z["pos"][:n])
            assert all(np.array_equal(x[key][:n][ox], z[key][:n][oz]) for key in ("k", "v", "word", "pos"))
    for g in (hst, sta):
        assert g.corm_cache_stats()["device_status"] == 0
        assert g.corm_cache_pool_usage(0)[0] == _pages_expected(g.corm_cache_live_lens(0))


def test_paged_layers_have_pools_of_their_own():
    """Three layers, each with its own pool, page tables and bitmap: stepping them in mixed order matches the oracle
    layer by layer, and a prompt pass on one layer returns that layer's pages only."""
    cfg = CONFIGS[2].with_(n_layers=3, n_q_heads=4, n_kv_heads=4, prompt_min=300, prompt_max=300, steps=40,
                           recent_r=32, dense_layers=1)
    gpu = make_gpu_cache(cfg, 1, 4, n_layers=3, pool_pages=64)
    orc = make_oracle(cfg, 1, 4, n_layers=3)
    datas = [generate(cfg, layer=l) for l in range(3)]
    dt = cfg.dtype
    for l in (2, 0, 1):
        d = datas[l]
        gpu.corm_compress_prompt(l, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
        orc.compress_prompt(l, d.k_prompt, d.v_prompt, d.q_last, d.prompt_lens)
    for s in range(cfg.steps):
        for l in (1, 2, 0):
            d = datas[l]
            a = gpu.corm_decode_step(l, to_dev(d.q[s], dt), to_dev(d.k_new[s], dt), to_dev(d.v_new[s], dt))
            o = orc.decode_step(l, d.q[s], d.k_new[s], d.v_new[s])
            assert np.abs(a.float().cpu().numpy() - o).max() <= OUT_TOL[dt]
    for l in range(3):
        assert_states_equal(gpu, orc, l, 1, 4, f"layer {l}")
        assert gpu.corm_cache_pool_usage(l) == (_pages_expected(orc.live_lens(l)), 64)
    before = [gpu.corm_cache_pool_usage(l)[0] for l in range(3)]
    d = datas[1]
    gpu.corm_compress_prompt(1, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
    after = [gpu.corm_cache_pool_usage(l)[0] for l in range(3)]
    assert after[0] == before[0] and after[2] == before[2]
    assert after[1] == _pages_expected(gpu.corm_cache_live_lens(1))
    assert gpu.corm_cache_stats()["device_status"] == 0


def test_exhausted_pool_is_reported_not_fatal():
    """alpha = 0 evicts nothing. Sixteen units of 60 keys hold two pages each, which is the whole 32-page pool. Slots
    60..63 still fit the second page; the append to slot 64 needs a third page, finds none, the status word says so
    and the units stay as they were."""
    cfg = CONFIGS[1].with_(prompt_min=60, prompt_max=60, steps=12, alpha=0.0, n_q_heads=16, n_kv_heads=16, dtype="bf16")
    data = generate(cfg)
    dt = cfg.dtype
    gpu = make_gpu_cache(cfg, 1, 16, pool_pages=32)         # 16 units x 2 pages: the pool is full after the prompt
    gpu.corm_compress_prompt(0, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    assert gpu.corm_cache_pool_usage(0) == (32, 32)
    for s in range(8):                                      # slots 60..63 fit the second page; slot 64 needs a third
        gpu.corm_decode_step(0, to_dev(data.q[s], dt), to_dev(data.k_new[s], dt), to_dev(data.v_new[s], dt))
    st = gpu.corm_cache_stats()
    assert st["device_status"] == 6 and (gpu.corm_cache_live_lens(0) == 64).all()
    assert gpu.corm_cache_pool_usage(0) == (32, 32)


def test_paged_arguments():
    from paper_2404_15949_b200.binding import CormError
    cfg = CONFIGS[1].with_(n_q_heads=2, n_kv_heads=2)
    for bad in (31, 33, -32):                               # not a multiple of 32 / negative
        with pytest.raises(CormError):
            make_gpu_cache(cfg, 1, 2, pool_pages=bad)
    with pytest.raises(CormError):
        make_gpu_cache(cfg, 40, 2, pool_pages=64)           # fewer pages than units
    assert make_gpu_cache(cfg, 1, 2).corm_cache_pool_usage(0) == (0, 0)
