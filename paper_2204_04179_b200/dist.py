"""Host-side logic of running the step on several GPUs (one process per GPU).

The step shards over histories: a rank runs the whole path (its own dedup included) on its own histories and
no stage exchanges data with another rank.  What ranks share is one all-reduce of the parameter gradients per
update (the paper trains with distributed data parallelism, Section 5.1) and bookkeeping: which histories or
which seeds belong to whom, the slowest rank's time, and the total of interactions processed.  These helpers
take the `torch.distributed` module (or None for a single process) so that they run on NCCL and on gloo alike.
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


def allreduce_weighted_mean(tensors, weight: float, dist=None) -> float:
    """In place, on every rank: t <- sum_r weight_r * t_r / sum_r weight_r for each tensor of `tensors`.

    Eq. 8's loss is a mean over the predictions of a batch, so a rank's gradient is the mean over ITS predictions;
    the gradient of the global batch is the mean of the ranks' gradients weighted by their prediction counts
    (shards of unequal size, or with different amounts of padding, would otherwise be over-weighted).  `weight` is
    this rank's count.  Returns the total weight.  One all-reduce per tensor, plus one for the weights."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(weight)
    tensors = list(tensors)
    dev = tensors[0].device if tensors else "cpu"
    w = torch.tensor([float(weight)], dtype=torch.float64, device=dev)
    dist.all_reduce(w, op=dist.ReduceOp.SUM)
    total = float(w.item())
    for t in tensors:
        t.mul_(float(weight) / total)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return total


class _DeviceBuffer:
    """A raw device allocation seen through the CUDA array interface, so that torch can wrap it without a copy."""

    def __init__(self, ptr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (int(n),), "typestr": "<f4", "data": (int(ptr), False), "version": 2}


def gradient_tensors(g):
    """The library context's two gradient buffers (encoder, task module) as torch tensors over the same memory."""
    import torch
    from . import binding
    out = []
    for module in (binding.GRAM_MODULE_CE, binding.GRAM_MODULE_TASK):
        ptr, n = g.grads_device(module)
        if n:
            out.append(torch.as_tensor(_DeviceBuffer(ptr, n), device="cuda"))
    return out


def n_predictions(shape, labels: np.ndarray) -> int:
    """Predictions Eq. 8 averages over in one batch: real positions of the histories (KT), users (NR)."""
    if shape.task == "kt":
        return int((np.asarray(labels) >= 0).sum())
    return int(np.asarray(labels).shape[0])


def allreduce_grads(g, n_pred: int, dist=None) -> float:
    """Averages both modules' gradients of a library context over the ranks, in place on the device (NCCL), weighted by
    each rank's number of predictions.  Call between gram_step (context created with defer_update) and
    gram_optimizer_step.  The step has synchronised its stream when it returns, so the buffers are complete."""
    return allreduce_weighted_mean(gradient_tensors(g), n_pred, dist)
