"""world_size-2 check (gloo, CPU) of the multi-GPU plan: shards are independent and reproducible, and the reported
whole-job throughput is the tokens of all ranks over the slowest rank's time."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2404_15949_b200.sharding import aggregate_throughput, shard_config
from paper_2404_15949_b200.workload import CONFIGS, generate, prompt_lens


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = shard_config(CONFIGS[3], rank, world)
    lens = prompt_lens(cfg)
    value, max_ms, total = aggregate_throughput(10.0 * (rank + 1), 32 * 100)
    out.put((rank, cfg.seed, lens.tolist(), value, max_ms, total))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_shards_and_aggregation():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, l0, v0, m0, t0), (r1, s1, l1, v1, m1, t1) = res
    assert (s0, s1) == (15949, 15950) and l0 != l1                 # different data per shard
    assert m0 == m1 == 20.0 and t0 == t1 == 6400                     # slowest rank's time, all ranks' tokens
    assert v0 == v1 == 6400 / 20e-3


def test_shard_is_reproducible_and_matches_single_gpu_generator():
    cfg = shard_config(CONFIGS[3], 1, 4)
    a = generate(cfg, seqs=[3], kv_heads=[5], n_steps=2)
    b = generate(CONFIGS[3].with_(seed=CONFIGS[3].seed + 1), seqs=[3], kv_heads=[5], n_steps=2)
    assert np.array_equal(a.k_prompt, b.k_prompt) and np.array_equal(a.q, b.q)


def test_aggregate_without_process_group_is_local():
    v, ms, n = aggregate_throughput(5.0, 1000)
    assert (v, ms, n) == (1000 / 5e-3, 5.0, 1000)
