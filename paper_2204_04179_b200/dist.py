"""Host-side logic of running the step on several GPUs (one process per GPU).

The step shards over histories: a rank runs the whole path (its own dedup included) on its own histories and
no stage exchanges data with another rank.  What ranks share is bookkeeping only: which histories or which
seeds belong to whom, the slowest rank's time, and the total of interactions processed.  These helpers take
the `torch.distributed` module (or None for a single process) so that they run on NCCL and on gloo alike.
"""
from __future__ import annotations

import numpy as np


def rank_seed(seed: int, rank: int) -> int:
    """Seed of a rank's own synthetic batches (weak scaling: every rank draws B histories of its own)."""
    return int(seed) + 7919 * int(rank)


def history_shard(n_histories: int, rank: int, world: int) -> slice:
    """Contiguous block of histories of `rank` when one global batch is split (strong scaling).
    Blocks differ in size by at most one and cover 0..n_histories-1 exactly once."""
    base, extra = divmod(int(n_histories), int(world))
    start = rank * base + min(rank, extra)
    return slice(start, start + base + (1 if rank < extra else 0))


def shard_batch(ids: np.ndarray, labels: np.ndarray, rank: int, world: int):
    """This rank's histories of a global batch ids/labels [B, L]."""
    s = history_shard(ids.shape[0], rank, world)
    return np.ascontiguousarray(ids[s]), np.ascontiguousarray(labels[s])


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's time: what a multi-GPU throughput is computed from."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist=None, device="cpu") -> float:
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(interactions_this_rank: float, ms_this_rank: float, dist=None, device="cpu") -> float:
    """Whole-job interactions per second: all ranks' interactions over the slowest rank's time."""
    total = sum_over_ranks(interactions_this_rank, dist, device)
    ms = max_over_ranks(ms_this_rank, dist, device)
    return total / (ms / 1e3)
