"""Replica bookkeeping for multi-GPU runs.

The prune step does not shard: every sequence is scored, selected and gathered on its own, there is
no exchange step.  N GPUs therefore run N independent replicas of the single-GPU library; the only
things the ranks share are a barrier around the timed region and the slowest rank's time.  These
helpers hold that (tiny) logic so that it can be exercised without GPUs (gloo, CPU tensors).
"""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The largest ``value`` over all ranks (``value`` itself when not distributed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_per_step_max: float, world: int) -> float:
    """Whole-job units per second of ``world`` replicas that each process ``units_per_rank`` per step,
    the step taking as long as the slowest rank needs."""
    return world * units_per_rank / (ms_per_step_max * 1e-3)


def split_sequences(n_sequences: int, world: int, rank: int) -> range:
    """Which sequences of a batch a rank takes when one batch is dealt out over the replicas
    (contiguous, sizes differing by at most one)."""
    lo = n_sequences * rank // world
    hi = n_sequences * (rank + 1) // world
    return range(lo, hi)
