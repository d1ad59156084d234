"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU oracle on the same seeded inputs and
compare them element by element (outputs within tolerance; registers, positions and rows bit-exact)."""
from __future__ import annotations

import numpy as np
import torch

OUT_TOL = {"f32": 2e-3, "bf16": 2e-2}     # max-abs tolerance on attention outputs, per cache dtype


def to_dev(a, dtype):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()


def make_gpu_cache(cfg, nb, nh, max_tokens=None, n_layers=1, pool_pages=0):
    from paper_2404_15949_b200.binding import CormCache
    return CormCache(n_layers, nb, nh * cfg.group, nh, cfg.head_dim, max_tokens or cfg.max_tokens, cfg.window_w,
                     cfg.recent_r, cfg.alpha, cfg.dtype, 0, pool_pages=pool_pages)


def make_oracle(cfg, nb, nh, max_tokens=None, n_layers=1):
    from oracle import CormOracle
    return CormOracle(n_layers, nb, nh * cfg.group, nh, cfg.head_dim, max_tokens or cfg.max_tokens, cfg.window_w,
                      cfg.recent_r, cfg.alpha)


def sorted_state(st):
    order = np.argsort(st["pos"], kind="stable")
    return dict(st, k=st["k"][order], v=st["v"][order], word=st["word"][order], pos=st["pos"][order])


def stamps_to_ages(stamps, n_tokens, w):
    """Registers of windows wider than 32 hold the step of the latest important verdict (0 = none). What Algorithm 1
    can still see of a register is how many queries ago that was, if fewer than w: the form the oracle reports."""
    age = n_tokens - stamps.astype(np.int64)
    return np.where((stamps != 0) & (age < w), age, -1).astype(np.int32)


def ages_to_stamps(ages, n_tokens):
    return np.where(ages >= 0, n_tokens - ages, 0).astype(np.uint32)


def assert_states_equal(gpu, orc, layer, nb, nh, tag=""):
    for b in range(nb):
        for h in range(nh):
            g = sorted_state(gpu.corm_cache_export_state(layer, b, h))
            o = orc.export_unit(layer, b, h)
            where = f"{tag} unit (b={b}, h={h})"
            assert g["live_len"] == o["live_len"], f"{where}: live {g['live_len']} != {o['live_len']}"
            assert len(set(g["pos"].tolist())) == g["live_len"], f"{where}: duplicate positions"
            assert np.array_equal(g["pos"], o["pos"]), f"{where}: live-index lists differ"
            if orc.w <= 32:
                assert np.array_equal(g["word"], o["word"]), f"{where}: verdict registers differ"
            else:
                assert np.array_equal(stamps_to_ages(g["word"], g["n_tokens"], orc.w), o["age"]), \
                    f"{where}: verdict registers differ"
            assert np.array_equal(g["k"].astype(np.float64), o["k"]), f"{where}: key rows differ"
            assert np.array_equal(g["v"].astype(np.float64), o["v"]), f"{where}: value rows differ"
            assert g["n_tokens"] == o["n_tokens"] and g["n_obs"] == o["n_obs"], where


def run_free(cfg, data, gpu, orc, layer=0, check_every=1, steps=None):
    """Prompt pass then decode steps on both sides with no resynchronisation. Returns max |out_gpu - out_oracle|."""
    nb, nh = len(data.seqs), len(data.kv_heads)
    dt = cfg.dtype
    gpu.corm_compress_prompt(layer, to_dev(data.k_prompt, dt), to_dev(data.v_prompt, dt), to_dev(data.q_last, dt),
                             data.prompt_lens)
    orc.compress_prompt(layer, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    assert_states_equal(gpu, orc, layer, nb, nh, "after prompt")
    worst = 0.0
    steps = data.n_steps if steps is None else steps
    q_d, k_d, v_d = to_dev(data.q[:steps], dt), to_dev(data.k_new[:steps], dt), to_dev(data.v_new[:steps], dt)
    for s in range(steps):
        out_g = gpu.corm_decode_step(layer, q_d[s], k_d[s], v_d[s]).float().cpu().numpy().astype(np.float64)
        out_o = orc.decode_step(layer, data.q[s], data.k_new[s], data.v_new[s])
        err = float(np.abs(out_g - out_o).max())
        worst = max(worst, err)
        assert err <= OUT_TOL[dt], f"step {s}: |out - oracle| = {err}"
        if (s + 1) % check_every == 0 or s == steps - 1:
            assert_states_equal(gpu, orc, layer, nb, nh, f"after step {s}")
    st = gpu.corm_cache_stats()
    assert st["device_status"] == 0
    if gpu.cfg.n_layers == 1:           # Section 3.1's sparsity counters: keys judged important / keys judged
        assert (st["important_keys"], st["attended_keys"]) == orc.sparsity()
    return worst
