#!/usr/bin/env python
"""Benchmark of the fused CORM decode+evict step (one JSON line on stdout).

A "step" is one decode step of the whole batch through every layer of the configuration (one layer for the default
workload): append, attention over every unit's live keys, verdicts, register update and compaction, one kernel
launch per layer. Default workload: the batched-throughput
configuration (batch 32, 32 heads, head_dim 128, bf16, ragged prompts in [2048, 4096]); the grouped-query workload is
measured as well and reported under `also`. Every workload is timed `--repeats` times over the same decode steps,
each pass from the restored post-prompt state, and the median pass is reported; the end-to-end figure (host buffers
through corm_decode_step_host) runs over the same steps from the same state.

    python bench.py --gpus 1 --steps 256 --warmup 16
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...   (independent shards)
    python bench.py --impl reference      (the CPU oracle timed on the host cores: a baseline, not the target)
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2404_15949_b200.workload import CONFIGS, generate  # noqa: E402

METRIC = "corm_decode_step_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of the dominant kernel per launch as ncu counted it, keyed by workload name; None until the counters are
# taken on the kernel as it stands now (a figure from an older kernel or another launch shape would mislead).
DRAM_TRAFFIC_BYTES_PER_LAUNCH = {}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Polls NVML (read-only) for SM clock and throttle reasons while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag, self.max_mhz = index, [], set(), False, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report that instead of guessing
            self.nv, self.err = None, repr(e)

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80}
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def result(self):
        if self.nv is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml_unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def algorithmic_bytes(cfg, attended, moved, unit_steps):
    """Bytes the method itself must move: live K+V once, register read+write, q+out, the appended row (read and
    written), and the rows compaction copies (read and written, with their register and position)."""
    e = 2 if cfg.dtype == "bf16" else 4
    d, G = cfg.head_dim, cfg.group
    return (attended * (2 * d * e + 8) + unit_steps * (2 * G * d * e + 4 * d * e) + moved * 2 * (2 * d * e + 8))


def oracle_baseline(cfg, n_seqs, n_steps):
    """The CPU oracle, as it stands, on a bounded sample of the same workload: the first n_seqs sequences (all
    heads), n_steps decode steps from the post-prompt-compression state."""
    from oracle import CormOracle
    seqs = list(range(min(n_seqs, cfg.batch)))
    n_steps = min(n_steps, cfg.steps)
    data = generate(cfg, seqs=seqs, n_steps=n_steps)
    orc = CormOracle(1, len(seqs), cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.max_tokens, cfg.window_w,
                     cfg.recent_r, cfg.alpha)
    orc.compress_prompt(0, data.k_prompt, data.v_prompt, data.q_last, data.prompt_lens)
    t0 = time.perf_counter()
    for s in range(n_steps):
        orc.decode_step(0, data.q[s], data.k_new[s], data.v_new[s])
    dt = time.perf_counter() - t0
    cores = os.cpu_count() or 1
    threads = min(cores, len(seqs) * cfg.n_kv_heads, int(os.environ.get("OMP_NUM_THREADS", cores)))
    return {"value": len(seqs) * n_steps / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{len(seqs)} of {cfg.batch} sequences x {cfg.n_kv_heads} kv heads, {n_steps} decode steps "
                      f"after prompt compression, fp64, OpenMP over units ({dt:.1f} s)"}, dt


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step, total = [], 0.0
    base = None
    for _ in range(args.warmup + args.steps):
        base, dt = oracle_baseline(cfg, args.ref_seqs, args.ref_steps)
        per_step.append(dt)
        total += dt
        if total > 150:      # keep the whole run within a few minutes
            break
    timed = per_step[min(args.warmup, len(per_step) - 1):]
    value = min(args.ref_seqs, cfg.batch) * min(args.ref_steps, cfg.steps) / float(np.mean(timed))
    base["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(timed), "warmup": len(per_step) - len(timed), "ms_per_step": 1e3 * float(np.mean(timed)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, args), "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(cfg, args, which=None):
    which = args.workload if which is None else which
    return {"workload": f"{cfg.name} (workload {which} of 5, configs[{which - 1}])", "batch": cfg.batch,
            "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
            "prompt_len": [cfg.prompt_min, cfg.prompt_max], "window_w": cfg.window_w, "recent_r": cfg.recent_r,
            "alpha": cfg.alpha, "layers_per_step": cfg.n_layers, "seed": cfg.seed,
            "l2": "live K/V read per step exceeds the 126 MB L2 (no flush needed)"}


def measure_workload(cfg, args, local, world, rank, want_e2e, want_clocks):
    """Prompt pass, then `repeats` timed passes over the same decode steps, each from the restored post-prompt state
    (the prompt pass is run again and the warm-up replayed), and an end-to-end pass over the same steps through the
    host-buffer entry point. Returns a dict of this rank's and the job's figures."""
    import torch
    import torch.distributed as dist
    from paper_2404_15949_b200.binding import CormCache
    from paper_2404_15949_b200.sharding import aggregate_throughput, shard_config

    cfg_r = shard_config(cfg, rank, world)              # each rank owns an independent shard: no data-path collective
    n_steps = args.warmup + args.steps
    cfg_r = cfg_r.with_(steps=max(cfg.steps, n_steps))
    L = cfg.n_layers                                    # a step = one token through every layer of the configuration
    t0 = time.perf_counter()
    data = [generate(cfg_r, layer=l, n_steps=n_steps) for l in range(L)]
    log(f"[rank {rank}] generated {cfg.name} inputs ({L} layer(s)) in {time.perf_counter() - t0:.1f} s")
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    dev = lambda a: torch.from_numpy(a).cuda().to(tdt).contiguous()
    cache = CormCache(L, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg_r.max_tokens, cfg.window_w,
                      cfg.recent_r, cfg.alpha, cfg.dtype, local, pool_pages=args.pool_pages)
    cache.corm_cache_set_tuning(args.split_len, 0 if args.no_fast else {"auto": 1, "inline": 2, "verdict": 3, "balanced": 4, "balanced-verdict": 5, "units": 6}[args.finish])
    ev = lambda: torch.cuda.Event(enable_timing=True)
    a, b = ev(), ev()
    prompts = [(dev(d.k_prompt), dev(d.v_prompt), dev(d.q_last), d.prompt_lens) for d in data]
    # [step][layer][...]: the layers' inputs of a step are contiguous, so that a configuration of several layers can be
    # stepped by one launch (corm_decode_step_layers)
    q_all = torch.stack([dev(d.q) for d in data], dim=1).contiguous()
    k_all = torch.stack([dev(d.k_new) for d in data], dim=1).contiguous()
    v_all = torch.stack([dev(d.v_new) for d in data], dim=1).contiguous()
    q_d = [q_all[:, l] for l in range(L)]
    k_d = [k_all[:, l] for l in range(L)]
    v_d = [v_all[:, l] for l in range(L)]
    out_all = torch.empty_like(q_all[0])
    out = out_all[0]
    # per-step views made once: slicing a tensor costs the host several microseconds, as much as a launch
    views = [[(q_all[s, l], k_all[s, l], v_all[s, l]) for l in range(L)] for s in range(n_steps)]

    def restore():
        """Back to the state right after the prompt pass. Returns the pass's device time (ms)."""
        torch.cuda.synchronize()
        a.record()
        for l in range(L):
            cache.corm_compress_prompt(l, *prompts[l])
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    # configurations of several layers step them all from one host call; the address tables are built once
    outs = [out_all[l] for l in range(L)]
    if L > 1:
        tabs = [tuple(cache.pointer_table([views[s][l][i] for l in range(L)], "q" if i == 0 else "kv") for i in range(3))
                for s in range(n_steps)]
        out_tab = cache.pointer_table(outs, "q")

    def step(s):
        if L > 1:
            cache.corm_decode_step_layers(0, tabs[s][0], tabs[s][1], tabs[s][2], out_tab)
        else:
            qv, kv, vv = views[s][0]
            cache.corm_decode_step(0, qv, kv, vv, out)

    out_steps = torch.empty_like(q_all) if args.api == "steps" else None

    def run(s0, s1, api):
        """Enqueue decode steps [s0, s1): one corm_decode_steps call, or one call per step."""
        if s1 <= s0:
            return
        if api == "steps":
            cache.corm_decode_steps(0, L, q_all[s0:s1], k_all[s0:s1], v_all[s0:s1], out_steps[s0:s1])
        else:
            for s in range(s0, s1):
                step(s)

    restore()                                            # untimed: the first launches load the kernels
    passes, prompt_ms, sampler = [], 0.0, None
    # with --api steps one more pass times the same steps through one call per step, reported as `per_step_calls`
    plan = [args.api] * args.repeats + (["step"] if args.api == "steps" else [])
    for rep, api in enumerate(plan):
        prompt_ms = restore()
        st0 = cache.corm_cache_stats()
        run(0, args.warmup, api)
        torch.cuda.synchronize()
        st1 = cache.corm_cache_stats()
        launches0 = cache.corm_cache_kernel_launches()
        if want_clocks and rep == 0:
            sampler = ClockSampler(local)
            sampler.start()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        a.record()
        t_issue = time.perf_counter()
        chained0 = cache.corm_cache_chained_launches()
        run(args.warmup, n_steps, api)
        b.record()
        issue_ms = 1e3 * (time.perf_counter() - t_issue)  # host time to enqueue the timed steps
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        st2 = cache.corm_cache_stats()
        passes.append(dict(ms=a.elapsed_time(b), issue_ms=issue_ms, st0=st0, st1=st1, st2=st2,
                           launches=cache.corm_cache_kernel_launches() - launches0,
                           chained=cache.corm_cache_chained_launches() - chained0))
    per_step_pass = passes.pop() if args.api == "steps" else None
    passes_sorted = sorted(passes, key=lambda x: x["ms"])
    med = passes_sorted[len(passes_sorted) // 2]

    # end to end through the host-buffer entry point, over the SAME steps from the same restored state: pinned inputs
    # read and the output written across the bus every step
    e2e_ms, h2d, d2h = None, 0, 0
    if want_e2e:
        pin = lambda t: t.contiguous().cpu().pin_memory()
        qh = [pin(x) for x in q_d]
        kh = [pin(x) for x in k_d]
        vh = [pin(x) for x in v_d]
        oh = torch.empty_like(qh[0][0]).pin_memory()
        h2d = L * (qh[0][0].numel() + 2 * kh[0][0].numel()) * oh.element_size()
        d2h = L * oh.numel() * oh.element_size()
        hviews = [[(qh[l][s], kh[l][s], vh[l][s]) for l in range(L)] for s in range(n_steps)]
        if args.api == "steps":
            qs, ks, vs = pin(q_all), pin(k_all), pin(v_all)
            os_ = torch.empty_like(qs).pin_memory()

        def run_host(s0, s1):
            if s1 <= s0:
                return
            if args.api == "steps":
                cache.corm_decode_steps_host(0, L, qs[s0:s1], ks[s0:s1], vs[s0:s1], os_[s0:s1])
            else:
                for s in range(s0, s1):
                    for l in range(L):
                        cache.corm_decode_step_host(l, *hviews[s][l], oh)

        restore()
        run_host(0, args.warmup)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        a.record()
        run_host(args.warmup, n_steps)
        b.record()
        torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(b)
    if sampler is not None:
        sampler.stop_flag = True
        sampler.join()
    st3 = cache.corm_cache_stats()
    assert st3["device_status"] == 0, f"device status {st3['device_status']}"

    value, ms_max, _ = aggregate_throughput(med["ms"], cfg.batch * args.steps, "cuda")
    e2e_value = aggregate_throughput(e2e_ms, cfg.batch * args.steps, "cuda")[0] if e2e_ms else None
    unit_steps = L * cfg.batch * cfg.n_kv_heads * args.steps
    attended = med["st2"]["attended_keys"] - med["st1"]["attended_keys"]
    moved = med["st2"]["moved_rows"] - med["st1"]["moved_rows"]
    abytes = algorithmic_bytes(cfg, attended, moved, unit_steps)
    peak, peak_src = measured_peak()
    achieved = abytes / (med["ms"] * 1e-3) / 1e9
    launches_per_step = med["launches"] / (args.steps * L)
    traffic = DRAM_TRAFFIC_BYTES_PER_LAUNCH.get(cfg.name)
    res = {
        "value": value, "ms_per_step": ms_max / args.steps,
        "repeats": {"n": len(passes), "ms_per_step": [x["ms"] / args.steps for x in passes],
                    "spread": (passes_sorted[-1]["ms"] - passes_sorted[0]["ms"]) / med["ms"],
                    "reported": "median pass; every pass starts from the restored post-prompt state"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / 8000.0, "peak_source": peak_src, "traffic": traffic,
                     "traffic_note": None if traffic else "no ncu capture of the kernel as it stands at this launch shape",
                     "target": {"frac_of_nominal_8TBs": 0.60, "met": achieved / 8000.0 >= 0.60},
                     "kernel": ("decode_balanced_kernel" if launches_per_step < 1.5 and cfg.group > 1 and args.finish in ("auto", "balanced")
                                else "decode_fast_kernel") + f" ({launches_per_step:.2f} launches per layer per step, all counted in the time)",
                     "bytes_per_launch": abytes / (args.steps * L), "us_per_launch": 1e3 * med["ms"] / (args.steps * L)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": "the same decode steps as `value`, from the same restored state",
                "api": "corm_decode_steps_host" if args.api == "steps" else "corm_decode_step_host per step and layer"},
        "gpu_launches": med["launches"], "host_issue_us_per_step": 1e3 * med["issue_ms"] / args.steps,
        "api": ("corm_decode_steps: the timed steps enqueued by one call" if args.api == "steps" else
                "one corm_decode_step" + ("_layers" if L > 1 else "") + " call per step"),
        "chained_launches": med["chained"],
        "retention": med["st2"]["retention"],
        "live_keys_per_unit": med["st2"]["live_keys"] / (L * cfg.batch * cfg.n_kv_heads),
        "evicted_keys_timed": med["st2"]["evicted_keys"] - med["st1"]["evicted_keys"], "moved_rows_timed": moved,
        "important_key_fraction_timed": (med["st2"]["important_keys"] - med["st1"]["important_keys"]) / max(1, attended),
        "prompt_pass_ms": prompt_ms, "retention_after_prompt": med["st0"]["retention"],
        "near_threshold_prompt_pass": med["st0"]["near_threshold"],
        "arena_bytes": int(cache.arena.numel()),
    }
    if per_step_pass is not None:       # the same steps, one host call per step (no launch is chained to the one before)
        res["per_step_calls"] = {
            "value": aggregate_throughput(per_step_pass["ms"], cfg.batch * args.steps, "cuda")[0], "unit": UNIT,
            "ms_per_step": per_step_pass["ms"] / args.steps,
            "host_issue_us_per_step": 1e3 * per_step_pass["issue_ms"] / args.steps}
    if sampler is not None:
        res["clocks"] = sampler.result()
    if args.pool_pages:
        res["pool_pages_in_use"] = sum(cache.corm_cache_pool_usage(l)[0] for l in range(L))
        # the paper's own metric, made physical: K+V bytes of the pages held against K+V bytes of every token seen
        row = 2 * cfg.head_dim * (2 if cfg.dtype == "bf16" else 4)
        res["kv_bytes_held"] = res["pool_pages_in_use"] * 32 * row
        res["kv_bytes_full_cache"] = st3["appended_keys"] * row
        res["kv_memory_reduction"] = 1.0 - res["kv_bytes_held"] / max(1, res["kv_bytes_full_cache"])
    cache.close()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--api", default="steps", choices=["steps", "step"],
                    help="steps: the timed steps are enqueued by one corm_decode_steps call (consecutive launches chained "
                         "where the kernels allow it); step: one corm_decode_step / corm_decode_step_layers call per step")
    ap.add_argument("--repeats", type=int, default=3, help="timed passes over the same steps; the median is reported")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end pass through the host-buffer entry point")
    ap.add_argument("--e2e-steps", type=int, default=None, help="0 skips the end-to-end pass (same as --no-e2e)")
    ap.add_argument("--also", default="4", help="comma-separated workloads measured as well and reported under `also` "
                                                "(default: the grouped-query target workload); empty = none")
    ap.add_argument("--ref-seqs", type=int, default=32)
    ap.add_argument("--ref-steps", type=int, default=512)
    ap.add_argument("--split-len", type=int, default=0)
    ap.add_argument("--no-fast", action="store_true")
    ap.add_argument("--finish", default="auto", choices=["auto", "inline", "verdict", "balanced", "balanced-verdict", "units"],
                    help="which decode kernels: automatic, the block-per-split kernels finishing long units inside the "
                         "decode launch / by the verdict launch, or the balanced single-launch kernel")
    ap.add_argument("--alpha", type=float, default=None, help="override the threshold scale (0 keeps every key)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--window", type=int, default=None, help="override the verdict window w (1..256)")
    ap.add_argument("--recent", type=int, default=None, help="override the protected recent tokens r")
    ap.add_argument("--pool-pages", type=int, default=0,
                    help="paged cache with this many 32-key pages per layer (multiple of 32); 0 = one slab per unit")
    args = ap.parse_args()

    def configured(which):
        cfg = CONFIGS[which]
        if args.alpha is not None:
            cfg = cfg.with_(alpha=args.alpha, name=cfg.name + f"_alpha{args.alpha:g}")
        if args.window is not None:
            cfg = cfg.with_(window_w=args.window, name=cfg.name + f"_w{args.window}")
        if args.recent is not None:
            cfg = cfg.with_(recent_r=args.recent, name=cfg.name + f"_r{args.recent}")
        return cfg

    cfg = configured(args.workload)
    if args.impl == "reference":
        return run_reference(args, cfg)

    import torch
    import torch.distributed as dist

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; the CORM path has no CPU fallback"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    want_e2e = not args.no_e2e and args.e2e_steps != 0
    main_res = measure_workload(cfg, args, local, world, rank, want_e2e, True)
    also = []
    for w in [int(x) for x in args.also.split(",") if x.strip()]:
        if w == args.workload:
            continue
        cfg_w = configured(w)
        saved = args.steps
        args.steps = min(args.steps, cfg_w.steps - args.warmup) if cfg_w.steps > args.warmup else args.steps
        r = measure_workload(cfg_w, args, local, world, rank, False, False)
        keep = ("value", "ms_per_step", "repeats", "roofline", "gpu_launches", "host_issue_us_per_step", "retention",
                "live_keys_per_unit", "prompt_pass_ms", "api", "chained_launches", "per_step_calls")
        also.append(dict({"config": workload_config(cfg_w, args, w), "steps": args.steps, "unit": UNIT},
                         **{k: r[k] for k in keep}))
        args.steps = saved
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    line = {
        "metric": METRIC, "value": main_res.pop("value"), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": main_res.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 logits / f32 accumulation over " + cfg.dtype + " cache", "data": "synthetic",
        "config": workload_config(cfg, args, args.workload),
    }
    line.update(main_res)
    line["paper_context"] = "paper reports KV memory only: up to 70% reduction (V100-32GB / A100-80GB), no throughput"
    if args.pool_pages:
        line["config"]["pool_pages"] = args.pool_pages
    if also:
        line["also"] = also
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"], _ = oracle_baseline(cfg, args.ref_seqs, args.ref_steps)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
