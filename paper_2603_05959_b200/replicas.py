"""Host-side logic of the multi-GPU benchmark: the path shards only across independent streams (replicas, no
data-path collective).  Every rank runs its own stream of frames with its own seed; the job's rate is the frames of
all ranks divided by the slowest rank's device time."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's stream: distinct streams, reproducible per rank."""
    return int(base_seed) + int(rank)


def max_over_ranks(values_ms, world: int, device=None):
    """Element-wise maximum over the ranks of a list of per-rank times (milliseconds)."""
    if world <= 1:
        return [float(v) for v in values_ms]
    t = torch.tensor([float(v) for v in values_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def aggregate_rate(units_per_rank: int, time_ms: float, world: int) -> float:
    """Whole-job rate: units of all ranks / the (already maximal) time."""
    return world * units_per_rank / (time_ms * 1e-3)
