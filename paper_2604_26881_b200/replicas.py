"""Host-side logic of running the layer on several GPUs of one node.

The layer has no exchange step: tokens are independent, so every rank is a replica that works on
its own batch.  What the ranks share is only the timing protocol: a barrier on both sides of the
timed region, the maximum of the per-rank times, and the sum of the tokens processed.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch a rank generates: rank 0 keeps the base seed, the others get distinct ones."""
    return base_seed + rank


def barrier(world: int, device_sync=None) -> None:
    if world > 1:
        dist.barrier()
    if device_sync is not None:
        device_sync()


def max_over_ranks(values, world: int, device=None):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank decides)."""
    if world <= 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def sum_over_ranks(value: float, world: int, device=None) -> float:
    if world <= 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t[0])


def aggregate_throughput(tokens_this_rank: int, steps: int, ms_this_rank: float, world: int, device=None):
    """(tokens/s of the whole job, ms per step): all ranks' tokens over the slowest rank's time."""
    ms = max_over_ranks([ms_this_rank], world, device)[0]
    tokens = sum_over_ranks(float(tokens_this_rank) * steps, world, device)
    return tokens / (ms * 1e-3), ms / steps
