"""Multi-GPU plan of the CORM path: independent shards, no data-path collective.

Every unit (layer, sequence, kv head with its group of query heads) is independent of every other (Algorithm 1 runs
per head; sequences never interact), so N GPUs each own whole sequences with their own arena and step them without
exchanging anything. The only cross-rank traffic is the reduction of the timing / counters for reporting.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_config(cfg, rank: int, world: int):
    """Weak scaling: rank r steps its own batch of cfg.batch sequences, drawn from seed cfg.seed + r."""
    assert 0 <= rank < world
    return cfg.with_(seed=cfg.seed + rank)


def aggregate_throughput(local_ms: float, local_tokens: int, device="cpu"):
    """Whole-job tokens/s = tokens of all ranks / slowest rank's time. Returns (value, max_ms, total_tokens).
    Works on any initialised backend (nccl with a cuda device, gloo on cpu); without a process group it is local."""
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    n = torch.tensor([float(local_tokens)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    max_ms, total = float(t[0]), float(n[0])
    return total / (max_ms * 1e-3), max_ms, int(total)
