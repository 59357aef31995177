"""Host-side plumbing for running the step on several GPUs of one node.

The draft-and-verify step is independent per sequence (the paper's Sec. 3.3 describes one
sequence; nothing couples two of them), so several GPUs are used as replicas: every rank keeps
the weights, takes its own sequences and runs the same five calls.  There is no exchange step
and therefore no collective on the data path; the only communication is this bookkeeping
(a barrier around the timed region, the slowest rank's time, the launch count), which works
with any torch.distributed backend ("nccl" on GPUs, "gloo" on CPUs).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic sequences of `rank`: every rank drafts for its own sequences."""
    return int(base_seed) + int(rank)


def shard_sequences(n_sequences: int, rank: int, world: int) -> range:
    """Contiguous share of `n_sequences` global sequence ids owned by `rank` (sizes differ by
    at most one; every id is owned by exactly one rank)."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    lo = n_sequences * rank // world
    hi = n_sequences * (rank + 1) // world
    return range(lo, hi)


def _device_for_backend() -> torch.device:
    if dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def max_over_ranks(values: Sequence[float]) -> List[float]:
    """Element-wise maximum of per-rank timings (a multi-GPU time is the slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=_device_for_backend())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def sum_over_ranks(value: int) -> int:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(value)
    t = torch.tensor([int(value)], dtype=torch.int64, device=_device_for_backend())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def aggregate_throughput(steps_per_rank: int, ms_local: float) -> Tuple[float, float]:
    """Whole-job steps/s and the time it is based on: all ranks' steps over the slowest rank's
    time for the timed region."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    (ms,) = max_over_ranks([ms_local])
    return world * steps_per_rank / (ms * 1e-3), ms
