"""Several GPUs: independent replicas, no collective on the data path.

The streams of Algorithm 1 are independent (no step couples two utterances), so more GPUs means
more streams: every rank holds the weights, owns a share of the streams and runs the verify step on
them alone.  What the ranks exchange is bookkeeping only: a barrier before a timed region and the
slowest rank's time after it.  This module holds that bookkeeping, written against
`torch.distributed` so that it runs over NCCL on GPUs and over gloo in CPU tests.
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(world size, rank, local rank) as torchrun exports them; (1, 0, 0) outside torchrun."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def shard_streams(n_streams: int, world: int, rank: int) -> List[int]:
    """Streams of a job of `n_streams` that rank `rank` of `world` owns: round robin, so that
    ragged lengths sorted by arrival spread evenly.  Every stream has exactly one owner."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    return list(range(rank, n_streams, world))


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def slowest(times_ms: Sequence[float], world: int, device: torch.device) -> List[float]:
    """Element-wise maximum over the ranks of each rank's list of measured times."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def total(units: int, world: int, device: torch.device) -> int:
    """Sum over the ranks of the units (streams, steps, tokens) each one processed."""
    t = torch.tensor([units], dtype=torch.int64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t[0])


def job_rate(units_per_rank: int, elapsed_ms: float, world: int, device: torch.device) -> float:
    """Whole-job rate in units per second: the units of all ranks over the slowest rank's time."""
    worst = slowest([elapsed_ms], world, device)[0]
    return total(units_per_rank, world, device) / (worst * 1e-3)
