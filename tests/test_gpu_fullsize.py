"""Parity at the benchmark's full sizes and in its launch configuration (automatic tuning, fast path on), over
the configurations' whole horizons.

The CUDA library steps the whole configuration for every decode step it defines (256 / 512 / 256 / 1024); the CPU
oracle steps a sample of its units (they are independent, and the generator yields identical slices for any subset),
free-running from the prompt pass with no resynchronisation, once through one corm_decode_steps call per 32 steps
(the benchmark's calls) and once through one call per step. Outputs of the sampled units must agree within the
cache dtype's tolerance at every step; registers, positions and rows must be bit-exact every 32 steps and at the
end, with the library enqueued far ahead of the host in between, as in the benchmark. That reaches the launch shapes
the benchmark spends its time in: one block per unit on the batch-32 workload, the balanced kernel on the grouped
one, planted-key drift and continuous compaction on the long-context one.

The oracle's count of probabilities within 1e-6 (relative) of the threshold is zero on the samples fixed here
(chosen by scanning candidate units with the oracle alone) and asserted so, except for the 32k-token configuration:
there one unit makes 5e7 evaluations over its horizon, 2e6 in the prompt pass alone, at about one in-band evaluation
per 1.3e6, so no sample of it is free of them; the count is printed and parity is required in full, in-band keys
included.
"""
import numpy as np
import pytest
import torch

from paper_2404_15949_b200.workload import CONFIGS, generate
from parity_util import OUT_TOL, make_oracle, sorted_state, to_dev

pytestmark = pytest.mark.gpu

CASES = [
    # config, layers sampled, sequences sampled, kv heads sampled (per layer), expect zero near-threshold
    (3, [0], [0, 17], {0: [3, 9]}, True),
    (4, [0], [1, 5], {0: [4, 5]}, True),
    (2, [0, 5, 31], [0], {0: [0, 9], 5: [1, 8], 31: [0, 3]}, True),
    (5, [0], [0], {0: [0]}, False),
]
CHECK_EVERY = 32


@pytest.mark.parametrize("api", ["steps", "step"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: f"config{c[0]}")
def test_full_size_sampled_units(case, api):
    """api "steps": every layer of the configuration is stepped, 32 steps per corm_decode_steps call (what bench.py
    times: all layers of a step as one launch, launches chained); "step": one corm_decode_step call per step for the
    sampled layers."""
    from paper_2404_15949_b200.binding import CormCache
    which, layers, seqs, heads_by_layer, expect_zero_near = case
    cfg = CONFIGS[which]
    steps = cfg.steps
    G, dt = cfg.group, cfg.dtype
    gpu = CormCache(cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.max_tokens,
                    cfg.window_w, cfg.recent_r, cfg.alpha, dt, 0)           # default tuning = what bench.py times
    oracles, full, lens = {}, {}, {}
    stepped = list(range(cfg.n_layers)) if api == "steps" else layers
    for l in stepped:
        d = generate(cfg, layer=l, n_steps=steps)
        gpu.corm_compress_prompt(l, to_dev(d.k_prompt, dt), to_dev(d.v_prompt, dt), to_dev(d.q_last, dt), d.prompt_lens)
        d.k_prompt = d.v_prompt = None                          # the prompts of 32 layers would not fit the host
        full[l], lens[l] = d, d.prompt_lens
        if l not in layers:
            continue
        heads = heads_by_layer[l]
        sub = generate(cfg, layer=l, seqs=seqs, kv_heads=heads, n_steps=steps)
        orc = make_oracle(cfg, len(seqs), len(heads))
        orc.compress_prompt(0, sub.k_prompt, sub.v_prompt, sub.q_last, sub.prompt_lens)
        oracles[l] = (orc, sub, heads)

    def check_states(tag):
        for l in layers:
            orc, _, heads = oracles[l]
            for ib, b in enumerate(seqs):
                for ih, h in enumerate(heads):
                    g = sorted_state(gpu.corm_cache_export_state(l, b, h))
                    o = orc.export_unit(0, ib, ih)
                    where = f"{tag}: layer {l} seq {b} head {h}"
                    assert g["live_len"] == o["live_len"], where
                    assert np.array_equal(g["pos"], o["pos"]), where + " live-index list"
                    assert np.array_equal(g["word"], o["word"]), where + " registers"
                    assert np.array_equal(g["k"].astype(np.float64), o["k"]), where + " key rows"
                    assert np.array_equal(g["v"].astype(np.float64), o["v"]), where + " value rows"

    check_states("after prompt")
    worst = 0.0
    if api == "steps":                                          # [step][layer][...] as corm_decode_steps takes them
        q_all, k_all, v_all = (torch.stack([to_dev(getattr(full[l], name), dt) for l in stepped], dim=1).contiguous()
                               for name in ("q", "k_new", "v_new"))
    else:
        dev_in = {l: tuple(to_dev(a, dt) for a in (full[l].q, full[l].k_new, full[l].v_new)) for l in layers}
    for s0 in range(0, steps, CHECK_EVERY):
        chunk = range(s0, min(steps, s0 + CHECK_EVERY))
        if api == "steps":
            s1 = chunk[-1] + 1
            out_all = gpu.corm_decode_steps(0, cfg.n_layers, q_all[s0:s1], k_all[s0:s1], v_all[s0:s1])
            outs = {l: list(out_all[:, l]) for l in layers}
        else:
            outs = {l: [] for l in layers}
            for s in chunk:                                    # the library runs ahead of the host for a whole chunk
                for l in layers:
                    qd, kd, vd = dev_in[l]
                    outs[l].append(gpu.corm_decode_step(l, qd[s], kd[s], vd[s]))
        for l in layers:
            orc, sub, heads = oracles[l]
            got = torch.stack(outs[l]).float().cpu().numpy()
            for i, s in enumerate(chunk):
                ref = orc.decode_step(0, sub.q[s], sub.k_new[s], sub.v_new[s])
                for ib, b in enumerate(seqs):
                    for ih, h in enumerate(heads):
                        err = np.abs(got[i, b, h * G:(h + 1) * G] - ref[ib, ih * G:(ih + 1) * G]).max()
                        worst = max(worst, float(err))
                        assert err <= OUT_TOL[dt], (s, l, b, h, err)
        check_states(f"after step {chunk[-1]}")
    near = sum(o[0].counters()["near_threshold"] for o in oracles.values())
    print(f"config {which}: max |out - oracle| = {worst:.2e}, near-threshold evaluations in the sample = {near}")
    if expect_zero_near:
        assert near == 0
    st = gpu.corm_cache_stats()
    assert st["device_status"] == 0
    # properties that hold at any size: every unit keeps at least its recent window, never more than it was given
    for l in stepped:
        live = gpu.corm_cache_live_lens(l)
        seen = lens[l][:, None] + steps
        assert (live <= seen).all() and (live >= np.minimum(seen, cfg.recent_r)).all()
    if api == "steps" and which != 5:     # the launches were chained (the long-context units keep the verdict launch)
        assert gpu.corm_cache_chained_launches() >= steps // 2
