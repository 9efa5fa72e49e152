"""Multi-GPU plumbing: the path shards by sequence with no exchange step.

Every (sequence, KV head) pair is independent in both the append and the decode path, so N GPUs
run N disjoint batches (replicas of the tables, weak scaling) and nothing crosses NVLink on the
data path.  The only communication is the timing reduction of the benchmark (max over ranks).
"""
from __future__ import annotations

import numpy as np


def shard_sequences(n_seq: int, rank: int, world: int) -> np.ndarray:
    """Indices of the sequences rank `rank` owns when a global batch is split (contiguous blocks,
    sizes differ by at most one)."""
    base, rem = divmod(n_seq, world)
    start = rank * base + min(rank, rem)
    return np.arange(start, start + base + (1 if rank < rem else 0))


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over the default process group (a no-op without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
