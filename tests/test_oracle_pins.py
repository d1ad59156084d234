"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle itself.

Hand-worked cases (tests/golden), full attention at alpha = 0 against a library softmax, agreement with the
per-key verdict-history statement of the policy (oracle/verdict_history.py), brute force over all subsets on tiny inputs, closed-form special cases and
per-step invariants. A dropped term, wrong sign/index or transposed operand in the oracle fails at least one.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import CormOracle
from oracle.verdict_history import HistoryUnit

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line)
    return rows


def _logit_inputs(c, d=64):
    """q, k_j with q.k_j/sqrt(d) = ln c_j up to one float32 rounding; v_j = j in every channel."""
    q = np.zeros((d,), dtype=np.float32)
    q[0] = np.sqrt(d)
    k = np.zeros((len(c), d), dtype=np.float64)
    k[:, 0] = np.log(np.asarray(c, dtype=np.float64))
    v = np.tile(np.arange(1, len(c) + 1, dtype=np.float32)[:, None], (1, d))
    return q, k.astype(np.float32), v


def _empty_prompt(o, d):
    o.compress_prompt(0, np.zeros((o.B, o.Hkv, 0, d), np.float32), None, None, [0] * o.B)


def test_handworked_decode_case():
    rows = _read_golden("handworked_decode.txt")
    c = [int(x) for x in rows[0].split()[1:]]
    q, k, v = _logit_inputs(c)
    o = CormOracle(1, 1, 1, 1, 64, 16, 2, 1, 1.0)
    _empty_prompt(o, 64)
    for line in rows[1:]:
        t, live, out, words = [x.strip() for x in line.split("|")]
        t = int(t)
        got = o.decode_step(0, q[None, None], k[t - 1][None, None], v[t - 1][None, None])
        st = o.export_unit(0, 0, 0)
        assert st["pos"].tolist() == [int(x) for x in live.split()], (t, st["pos"])
        assert st["word"].tolist() == [int(x, 2) for x in words.split()], (t, st["word"])
        # float32 storage of ln c_j perturbs the logits by ~1e-7, hence the tolerance on the fraction
        assert np.allclose(got[0, 0], float(Fraction(out)), rtol=0, atol=2e-6), (t, got[0, 0, 0])
        assert st["n_tokens"] == t and st["n_obs"] == min(t, 2)


def test_handworked_prompt_case():
    rows = dict((r.split()[0], r.split()[1:]) for r in _read_golden("handworked_prompt.txt"))
    c = [int(x) for x in rows["c"]]
    q, k, v = _logit_inputs(c)
    o = CormOracle(1, 1, 1, 1, 64, 16, 2, 1, 1.0)
    q_last = np.stack([q, q])[None, None]                      # the two recorded queries are equal
    o.compress_prompt(0, k[None, None], v[None, None], q_last, [4])
    st = o.export_unit(0, 0, 0)
    assert st["pos"].tolist() == [int(x) for x in rows["live_after"]]
    assert st["word"].tolist() == [int(x, 2) for x in rows["words_after"]]
    # a window of 3 records positions 2,3,4: key1 111; key2 (1/9 < 1/2 at i=2, then minor twice) 000; key3 000;
    # key4 001 -> same survivors
    o2 = CormOracle(1, 1, 1, 1, 64, 16, 3, 1, 1.0)
    o2.compress_prompt(0, k[None, None], v[None, None], np.stack([q, q, q])[None, None], [4])
    st2 = o2.export_unit(0, 0, 0)
    assert st2["pos"].tolist() == [1, 4] and st2["word"].tolist() == [0b111, 0b001]
    # with a window not yet full (w=4 > 3 usable rows... P=4 gives 4 rows; use w=5) nothing is evicted and the
    # pre-eviction words of the two newest rows show in the low bits
    o3 = CormOracle(1, 1, 1, 1, 64, 16, 5, 1, 1.0)
    o3.compress_prompt(0, k[None, None], v[None, None], np.stack([q] * 5)[None, None], [4])
    st3 = o3.export_unit(0, 0, 0)
    assert st3["pos"].tolist() == [1, 2, 3, 4] and st3["n_obs"] == 4
    assert [int(x) & 3 for x in st3["word"]] == [int(x, 2) for x in rows["words_before_eviction"]]


def _random_case(rng, B, Hq, Hkv, d, P, steps, w, scale=1.5):
    G = Hq // Hkv
    k = rng.standard_normal((B, Hkv, P + steps, d)).astype(np.float32) * scale
    v = rng.standard_normal((B, Hkv, P + steps, d)).astype(np.float32)
    q = rng.standard_normal((B, Hq, w + steps, d)).astype(np.float32) * scale
    return k, v, q, G


@pytest.mark.parametrize("seed", range(6))
def test_alpha_zero_is_full_attention(seed):
    """alpha = 0 makes every key important, nothing is evicted, and each step is plain softmax(qK^T/sqrt(d))V over
    all tokens so far, checked against torch's softmax in fp64."""
    rng = np.random.default_rng(seed)
    B, Hq, Hkv, d, P, steps, w, r = 2, 4, 2, 8, 5, 12, 3, 2
    k, v, q, G = _random_case(rng, B, Hq, Hkv, d, P, steps, w)
    o = CormOracle(1, B, Hq, Hkv, d, P + steps, w, r, 0.0)
    o.compress_prompt(0, k[:, :, :P], v[:, :, :P], q[:, :, :w], [P] * B)
    for s in range(steps):
        out = o.decode_step(0, q[:, :, w + s], k[:, :, P + s], v[:, :, P + s])
        n = P + s + 1
        K = torch.from_numpy(k[:, :, :n]).double().repeat_interleave(G, dim=1)
        V = torch.from_numpy(v[:, :, :n]).double().repeat_interleave(G, dim=1)
        Q = torch.from_numpy(q[:, :, w + s]).double()
        ref = torch.einsum("bhn,bhnd->bhd", torch.softmax(torch.einsum("bhd,bhnd->bhn", Q, K) / d ** 0.5, -1), V)
        assert np.allclose(out, ref.numpy(), rtol=1e-12, atol=1e-12)
        assert (o.live_lens(0) == n).all()
    assert o.counters()["evicted"] == 0


@pytest.mark.parametrize("seed", range(40))
def test_shift_register_equals_verdict_history(seed):
    """C oracle (shift registers) against the per-key verdict histories on random tiny cases, prompt included."""
    rng = np.random.default_rng(1000 + seed)
    Hkv = int(rng.integers(1, 3))
    G = int(rng.integers(1, 4))
    Hq, B = Hkv * G, int(rng.integers(1, 3))
    d, w, r = int(rng.integers(1, 5)), int(rng.integers(1, 6)), int(rng.integers(1, 5))
    P, steps = int(rng.integers(0, 9)), int(rng.integers(4, 16))
    alpha = float(rng.choice([0.5, 1.0, 1.0, 2.0]))
    k, v, q, _ = _random_case(rng, B, Hq, Hkv, d, P, steps, w, scale=2.0)
    o = CormOracle(1, B, Hq, Hkv, d, P + steps, w, r, alpha)
    lens = [P] * B
    if B == 2 and P > 0:
        lens[1] = int(rng.integers(0, P + 1))                  # ragged prompts
    units = {}
    for b in range(B):
        for h in range(Hkv):
            u = HistoryUnit(d, w, r, alpha)
            u.compress_prompt(k[b, h, :lens[b]], v[b, h, :lens[b]], q[b, h * G:(h + 1) * G, :w])
            units[b, h] = u
    o.compress_prompt(0, k[:, :, :P], v[:, :, :P], q[:, :, :w], lens)
    for s in range(steps + 1):
        for b in range(B):
            for h in range(Hkv):
                st, u = o.export_unit(0, b, h), units[b, h]
                assert st["pos"].tolist() == u.pos.tolist(), (s, b, h)
                assert st["word"].tolist() == u.words().tolist(), (s, b, h)
                assert np.array_equal(st["k"], u.keys) and np.array_equal(st["v"], u.values)
        if s == steps:
            break
        k_new = np.stack([k[b, :, lens[b] + s] for b in range(B)])
        v_new = np.stack([v[b, :, lens[b] + s] for b in range(B)])
        out = o.decode_step(0, q[:, :, w + s], k_new, v_new)
        for b in range(B):
            for h in range(Hkv):
                ref = units[b, h].decode_step(q[b, h * G:(h + 1) * G, w + s], k_new[b, h], v_new[b, h])
                assert np.allclose(out[b, h * G:(h + 1) * G], ref, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("seed", range(10))
def test_wide_windows_equal_verdict_history(seed):
    """Windows beyond 32 queries (the paper's experiments use up to 256): multi-word registers against the per-key
    verdict histories, compared through the live lists and the age of each key's newest 'important' verdict."""
    rng = np.random.default_rng(3000 + seed)
    G = int(rng.integers(1, 3))
    d, w, r = 3, int(rng.choice([33, 40, 64, 65, 100])), int(rng.integers(1, 20))
    P, steps = int(rng.integers(0, 150)), int(rng.integers(40, 90))
    k, v, q, _ = _random_case(rng, 1, G, 1, d, P, steps, w, scale=2.5)
    o = CormOracle(1, 1, G, 1, d, P + steps, w, r, 1.0)
    u = HistoryUnit(d, w, r, 1.0)
    u.compress_prompt(k[0, 0, :P], v[0, 0, :P], q[0, :, :w])
    o.compress_prompt(0, k[:, :, :P], v[:, :, :P], q[:, :, :w], [P])
    evicted = False
    for s in range(steps + 1):
        st = o.export_unit(0, 0, 0)
        assert st["pos"].tolist() == u.pos.tolist(), s
        assert st["age"].tolist() == u.ages().tolist(), s
        if s == steps:
            break
        out = o.decode_step(0, q[:, :, w + s], k[:, :, P + s], v[:, :, P + s])
        ref = u.decode_step(q[0, :, w + s], k[0, 0, P + s], v[0, 0, P + s])
        assert np.allclose(out[0], ref, rtol=1e-12, atol=1e-13)
        evicted |= o.live_len(0, 0, 0) < P + s + 1
    assert evicted or P + steps < w


@pytest.mark.parametrize("seed", range(8))
def test_bruteforce_eviction_sets(seed):
    """t <= 16: verdicts recomputed with a library softmax, and the kept set identified by enumerating all subsets of
    the live keys for the one that satisfies 'kept <=> recent, or important for some query among the last w'
    (Definition 4.1 with the window of the Approach paragraph)."""
    rng = np.random.default_rng(2000 + seed)
    d, w, r, G = 3, int(rng.integers(1, 4)), int(rng.integers(1, 4)), int(rng.integers(1, 3))
    alpha, steps = 1.0, 16
    o = CormOracle(1, 1, G, 1, d, steps, w, r, alpha)
    _empty_prompt(o, d)
    k = (rng.standard_normal((steps, d)) * 2).astype(np.float32)
    v = rng.standard_normal((steps, d)).astype(np.float32)
    q = (rng.standard_normal((steps, G, d)) * 2).astype(np.float32)
    history = []                                               # per step: {pos: verdict}
    live = []                                                  # positions
    for t in range(1, steps + 1):
        live = live + [t]
        K = torch.tensor(np.stack([k[p - 1] for p in live])).double()
        verdict = {p: False for p in live}
        for g in range(G):
            prob = torch.softmax(K @ torch.tensor(q[t - 1, g]).double() / d ** 0.5, 0)
            assert abs(float(prob.sum()) - 1) < 1e-12
            for p, pr in zip(live, prob.tolist()):
                verdict[p] = verdict[p] or pr >= alpha / t
        history.append(verdict)
        _, imp = o.decode_step(0, q[t - 1][None], k[t - 1][None, None], v[t - 1][None, None], want_verdicts=True)
        assert imp[0, 0, :len(live)].tolist() == [int(verdict[p]) for p in live]
        if len(history) >= w:
            recent_rows = history[-w:]

            def needed(p):
                return p > t - r or any(row.get(p, False) for row in recent_rows)

            valid = [S for n in range(len(live) + 1) for S in itertools.combinations(live, n)
                     if all((p in S) == needed(p) for p in live)]
            assert len(valid) == 1
            live = list(valid[0])
        assert o.export_unit(0, 0, 0)["pos"].tolist() == live


def test_invariants_on_generated_workload():
    from paper_2404_15949_b200.workload import CONFIGS, generate
    cfg = CONFIGS[1].with_(prompt_min=96, prompt_max=96, steps=48, recent_r=16)
    g = generate(cfg)
    o = CormOracle(1, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.max_tokens, cfg.window_w,
                   cfg.recent_r, cfg.alpha)
    o.compress_prompt(0, g.k_prompt, g.v_prompt, g.q_last, g.prompt_lens)
    prev = {h: o.export_unit(0, 0, h) for h in range(cfg.n_kv_heads)}
    evicted_any = False
    for s in range(cfg.steps):
        t = 96 + s + 1
        o.decode_step(0, g.q[s], g.k_new[s], g.v_new[s])
        for h in range(cfg.n_kv_heads):
            st = o.export_unit(0, 0, h)
            pos = st["pos"]
            assert (np.diff(pos) > 0).all()                                  # order kept
            assert set(range(t - cfg.recent_r + 1, t + 1)) <= set(pos.tolist())  # recent r always live
            assert set(pos.tolist()) <= set(prev[h]["pos"].tolist()) | {t}   # eviction is permanent
            old = pos <= t - cfg.recent_r
            assert (st["word"][old] != 0).all()                              # survivors outside the window are needed
            assert st["live_len"] <= prev[h]["live_len"] + 1
            evicted_any |= st["live_len"] < prev[h]["live_len"] + 1
            prev[h] = st
    c = o.counters()
    assert evicted_any and c["appended"] - c["evicted"] == int(o.live_lens(0).sum())


def test_warmup_blocks_eviction_until_w_rows():
    rng = np.random.default_rng(7)
    d, w, r, steps = 4, 5, 1, 9
    o = CormOracle(1, 1, 1, 1, d, steps, w, r, 1.0)
    _empty_prompt(o, d)
    for t in range(1, steps + 1):
        o.decode_step(0, rng.standard_normal((1, 1, d)).astype(np.float32) * 3,
                      rng.standard_normal((1, 1, d)).astype(np.float32) * 3,
                      rng.standard_normal((1, 1, d)).astype(np.float32))
        if t < w:
            assert o.live_len(0, 0, 0) == t and o.n_obs(0, 0) == t
    assert o.n_obs(0, 0) == w and o.live_len(0, 0, 0) < steps


def test_identical_keys_are_never_minor():
    """All keys equal: every probability is exactly 1/l >= 1/t, so nothing can be evicted at alpha = 1."""
    d, steps = 4, 20
    o = CormOracle(1, 1, 1, 1, d, steps, 2, 1, 1.0)
    _empty_prompt(o, d)
    kv = np.ones((1, 1, d), np.float32)
    for t in range(1, steps + 1):
        out = o.decode_step(0, np.full((1, 1, d), 0.37, np.float32), kv, kv * t)
        assert o.live_len(0, 0, 0) == t
        assert np.allclose(out, (t + 1) / 2, rtol=1e-13)          # mean of 1..t


def test_dominant_key_leaves_only_itself_and_the_recent_window():
    d, w, r, steps = 8, 3, 4, 30
    o = CormOracle(1, 1, 1, 1, d, steps, w, r, 1.0)
    _empty_prompt(o, d)
    q = np.zeros((1, 1, d), np.float32)
    q[0, 0, 0] = np.sqrt(d)
    for t in range(1, steps + 1):
        k = np.zeros((1, 1, d), np.float32)
        k[0, 0, 0] = 40.0 if t == 2 else 0.0                      # logit +40 over the rest
        o.decode_step(0, q, k, np.ones((1, 1, d), np.float32))
        if t > r + w + 2:
            assert o.export_unit(0, 0, 0)["pos"].tolist() == [2] + list(range(t - r + 1, t + 1))


def test_group_of_identical_heads_equals_single_head_and_or_rule():
    rng = np.random.default_rng(11)
    d, w, r, P, steps = 6, 3, 2, 7, 14
    k, v, q, _ = _random_case(rng, 1, 1, 1, d, P, steps, w, scale=2.0)
    single = CormOracle(1, 1, 1, 1, d, P + steps, w, r, 1.0)
    group = CormOracle(1, 1, 3, 1, d, P + steps, w, r, 1.0)
    q3 = np.repeat(q, 3, axis=1)
    single.compress_prompt(0, k[:, :, :P], v[:, :, :P], q[:, :, :w], [P])
    group.compress_prompt(0, k[:, :, :P], v[:, :, :P], q3[:, :, :w], [P])
    for s in range(steps):
        a = single.decode_step(0, q[:, :, w + s], k[:, :, P + s], v[:, :, P + s])
        b = group.decode_step(0, q3[:, :, w + s], k[:, :, P + s], v[:, :, P + s])
        assert np.array_equal(np.repeat(a, 3, axis=1), b)
        sa, sb = single.export_unit(0, 0, 0), group.export_unit(0, 0, 0)
        assert sa["pos"].tolist() == sb["pos"].tolist() and sa["word"].tolist() == sb["word"].tolist()
    # OR rule: a group's verdict is the union of what each head alone would say on the same cache
    two = CormOracle(1, 1, 2, 1, d, 4, 8, 8, 1.0)
    ones = [CormOracle(1, 1, 1, 1, d, 4, 8, 8, 1.0) for _ in range(2)]
    for o in [two] + ones:
        _empty_prompt(o, d)
    qq = (rng.standard_normal((4, 1, 2, d)) * 3).astype(np.float32)
    for t in range(4):
        kn, vn = k[:, :, t], v[:, :, t]
        _, imp = two.decode_step(0, qq[t], kn, vn, want_verdicts=True)
        sep = [o.decode_step(0, qq[t][:, g:g + 1], kn, vn, want_verdicts=True)[1] for g, o in enumerate(ones)]
        assert np.array_equal(imp, sep[0] | sep[1])


def test_positive_query_scaling_keeps_the_ranking():
    """Eq. 4: q and m*q (m > 0) rank the keys identically, so their important sets are nested."""
    rng = np.random.default_rng(5)
    d, n = 8, 12
    k = rng.standard_normal((n, d)).astype(np.float32) * 2
    q = rng.standard_normal((d,)).astype(np.float32)
    sets = []
    for m in (0.25, 1.0, 3.0):
        o = CormOracle(1, 1, 1, 1, d, n, 32, 32, 1.0)
        _empty_prompt(o, d)
        for j in range(n - 1):                                      # fill the cache (r = 32: no evictions)
            o.decode_step(0, np.zeros((1, 1, d), np.float32), k[j][None, None], k[j][None, None])
        _, imp = o.decode_step(0, (m * q)[None, None], k[n - 1][None, None], k[n - 1][None, None], want_verdicts=True)
        sets.append(set(np.nonzero(imp[0, 0])[0].tolist()))
    ranked = sorted(sets, key=len)
    assert ranked[0] <= ranked[1] <= ranked[2] and len(ranked[2]) >= 1


def test_near_threshold_band_counter():
    """Keys sitting exactly on the threshold (identical keys, l = t) are counted inside the band."""
    d = 4
    o = CormOracle(1, 1, 1, 1, d, 8, 2, 1, 1.0)
    _empty_prompt(o, d)
    kv = np.ones((1, 1, d), np.float32)
    for _ in range(5):
        o.decode_step(0, kv, kv, kv)
    c = o.counters()
    assert c["near_threshold"] == c["verdict_evals"] == 1 + 2 + 3 + 4 + 5


def test_near_band_width_follows_the_handworked_probabilities():
    """The counter of verdict evaluations with |p - alpha/t| <= rel * alpha/t, on the hand-worked decode case where every
    probability is known as a fraction (tests/golden/handworked_decode.txt): the expected counts are taken from those
    fractions here, for several band widths."""
    from fractions import Fraction as Fr
    c = [8, 1, 1, 4, 1, 1]
    live_before = [[1], [1, 2], [1, 2, 3], [1, 3, 4], [1, 4, 5], [1, 4, 5, 6]]     # keys attended at t = 1..6 (golden file)
    dist = []                                                   # |p - 1/t| / (1/t) of every evaluation, exactly
    for t, live in enumerate(live_before, start=1):
        Z = sum(c[j - 1] for j in live)
        dist += [abs(Fr(c[j - 1], Z) * t - 1) for j in live]
    for rel in (Fr(0), Fr(1, 10), Fr(1, 2), Fr(13, 20), Fr(3, 2), Fr(100)):
        o = CormOracle(1, 1, 1, 1, 64, 8, 2, 1, 1.0)
        o.set_near_band(float(rel))
        _empty_prompt(o, 64)
        q = np.zeros((1, 1, 64), np.float32); q[0, 0, 0] = 8.0
        for j in range(6):
            k = np.zeros((1, 1, 64), np.float32); k[0, 0, 0] = np.float32(np.log(c[j]))
            o.decode_step(0, q, k, np.full((1, 1, 64), j + 1.0, np.float32))
        n = o.counters()
        assert n["verdict_evals"] == len(dist) == 16
        # float32 ln(c_j) moves a probability by ~1e-7 relative: widths are chosen away from every exact distance
        assert all(abs(float(x - rel)) > 1e-3 for x in dist if x != 0)
        assert n["near_threshold"] == sum(1 for x in dist if x <= rel), float(rel)


@pytest.mark.parametrize("w,G", [(8, 1), (5, 2), (40, 1), (100, 2)])
def test_export_import_roundtrip_then_identical_future(w, G):
    from paper_2404_15949_b200.workload import CONFIGS, generate
    """A unit exported in mid-run (whole registers) and imported into a fresh oracle must have the same future:
    identical outputs, registers, positions and rows for the next 20 steps. One-word import is for windows of up
    to 32 queries and is refused beyond."""
    cfg = CONFIGS[1].with_(batch=2, n_q_heads=2 * G, n_kv_heads=2, head_dim=16, prompt_min=max(40, w + 5),
                           prompt_max=max(40, w + 5) + 30, steps=45, window_w=w, recent_r=6, alpha=2.0 if w > 32 else 1.0, gqa_rho=0.7 if G > 1 else 0.0,
                           hh_min=2, hh_max=4, seed=99)
    data = generate(cfg)
    mk = lambda: CormOracle(1, 2, 2 * G, 2, 16, cfg.max_tokens, w, 6, cfg.alpha)
    a, b = mk(), mk()
    a.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    for s in range(25):
        a.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
    assert a.counters()["evicted"] > 0
    b.compress_prompt(0, None, None, None, np.zeros(2, np.int32))                  # a fresh, empty cache
    for ib in range(2):
        for ih in range(2):
            st = a.export_unit(0, ib, ih)
            b.import_unit(0, ib, ih, st["k"], st["v"], st["regs"], st["pos"], st["n_tokens"], st["n_obs"])
            if w > 32:
                with pytest.raises(RuntimeError):
                    mk().import_unit(0, ib, ih, st["k"], st["v"], st["word"], st["pos"], st["n_tokens"], st["n_obs"])
    if w <= 32:                                                                      # the one-word form carries the same state
        c = mk()
        c.compress_prompt(0, None, None, None, np.zeros(2, np.int32))
        for ib in range(2):
            for ih in range(2):
                st = a.export_unit(0, ib, ih)
                c.import_unit(0, ib, ih, st["k"], st["v"], st["word"], st["pos"], st["n_tokens"], st["n_obs"])
    others = [b] + ([c] if w <= 32 else [])
    for s in range(25, 45):
        ref = a.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
        for o in others:
            assert np.array_equal(ref, o.decode_step(0, data.q[s], data.k_new[s], data.v_new[s]))
            for ib in range(2):
                for ih in range(2):
                    x, y = a.export_unit(0, ib, ih), o.export_unit(0, ib, ih)
                    for key in ("k", "v", "regs", "pos", "age", "live_len", "n_tokens", "n_obs"):
                        assert np.array_equal(x[key], y[key]), (s, ib, ih, key)


def test_bad_arguments_and_capacity():
    with pytest.raises(ValueError):
        CormOracle(1, 1, 3, 2, 4, 8, 2, 1, 1.0)
    with pytest.raises(ValueError):
        CormOracle(1, 1, 1, 1, 4, 8, 2, 0, 1.0)                 # r = 0 is rejected (the slice [-0:] selects everything)
    o = CormOracle(1, 1, 1, 1, 4, 2, 2, 1, 0.0)
    _empty_prompt(o, 4)
    x = np.ones((1, 1, 4), np.float32)
    o.decode_step(0, x, x, x)
    o.decode_step(0, x, x, x)
    with pytest.raises(RuntimeError):
        o.decode_step(0, x, x, x)


def test_sparsity_counters_match_the_verdict_rows():
    """The proportion of important keys (Section 3.1) is counted over decode steps: the counters must equal what the
    per-step verdict rows add up to, and with alpha = 0 every judged key is important."""
    from oracle import CormOracle
    rng = np.random.default_rng(5)
    for alpha in (1.0, 0.0):
        o = CormOracle(1, 2, 4, 2, 8, 64, 3, 2, alpha)
        kp = rng.standard_normal((2, 2, 10, 8)).astype(np.float32)
        vp = rng.standard_normal((2, 2, 10, 8)).astype(np.float32)
        ql = rng.standard_normal((2, 4, 3, 8)).astype(np.float32)
        o.compress_prompt(0, kp, vp, ql, np.array([10, 7], dtype=np.int32))
        assert o.sparsity() == (0, 0)                      # the prompt pass is not counted
        imp_sum = judged = 0
        for s in range(12):
            lens = o.live_lens(0)
            q = rng.standard_normal((2, 4, 8)).astype(np.float32) * 2
            kn = rng.standard_normal((2, 2, 8)).astype(np.float32)
            vn = rng.standard_normal((2, 2, 8)).astype(np.float32)
            _, imp = o.decode_step(0, q, kn, vn, want_verdicts=True)
            for b in range(2):
                for h in range(2):
                    imp_sum += int(imp[b, h, :lens[b, h] + 1].sum())
                    judged += int(lens[b, h]) + 1
        assert o.sparsity() == (imp_sum, judged)
        if alpha == 0.0:
            assert imp_sum == judged
        else:
            assert 0 < imp_sum < judged


def test_adjacent_query_similarity_closed_forms():
    """Eq. 3 between consecutive decode queries: a query repeated up to a positive factor gives 1, its negative -1, an
    orthogonal one 0, and random ones what numpy's dot and norms give; the first step after a prompt has no partner."""
    from oracle import CormOracle
    rng = np.random.default_rng(11)
    o = CormOracle(1, 1, 2, 2, 8, 64, 3, 2, 1.0)
    z = np.zeros((1, 2, 4, 8), dtype=np.float32)
    o.compress_prompt(0, rng.standard_normal((1, 2, 4, 8)).astype(np.float32), z.copy(), np.zeros((1, 2, 3, 8), dtype=np.float32),
                      np.array([4], dtype=np.int32))
    kn = rng.standard_normal((1, 2, 8)).astype(np.float32)
    q0 = rng.standard_normal((1, 2, 8)).astype(np.float32)
    e0 = np.zeros((1, 2, 8), dtype=np.float32); e0[..., 0] = 1
    e1 = np.zeros((1, 2, 8), dtype=np.float32); e1[..., 1] = 3
    qs = [q0, 2.5 * q0, -q0, e0, e1, q0, rng.standard_normal((1, 2, 8)).astype(np.float32)]
    expect, total = [None, 1.0, -1.0, None, 0.0, None, None], 0.0
    for i, q in enumerate(qs):
        before = o.similarity()
        o.decode_step(0, q, kn, kn)
        after = o.similarity()
        if i == 0:
            assert after == (0.0, 0)
            continue
        a, b = qs[i].astype(np.float64), qs[i - 1].astype(np.float64)
        ref = sum(float(a[0, h] @ b[0, h]) / (np.linalg.norm(a[0, h]) * np.linalg.norm(b[0, h])) for h in range(2))
        assert after[1] == before[1] + 2 and abs((after[0] - before[0]) - ref) < 1e-12
        if expect[i] is not None:
            assert abs((after[0] - before[0]) - 2 * expect[i]) < 1e-12
