"""Host-side logic of multi-GPU runs.  The sampling path does not shard across GPUs (a step is a latency chain
that needs the whole state twice); several GPUs run independent replicas -- different streams of the same workload,
one process per GPU, no collective on the data path.  What the ranks share is only the timing protocol: a barrier
on both sides of the timed region, the maximum of the per-rank device times, and the sum of the units produced.
"""
from __future__ import annotations

import os
from typing import Tuple


def rank_env() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) for a plain run."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def rank_seed(base_seed: int, rank: int) -> int:
    """Sampling seed of a replica: every rank draws its own streams."""
    return int(base_seed) + int(rank)


def init(backend: str, device=None):
    """Join the process group when the launcher started more than one rank; returns torch.distributed or None."""
    rank, world, _ = rank_env()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        if device is not None and backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
    return dist


def barrier(dist) -> None:
    if dist is not None:
        dist.barrier()


def max_over_ranks(value: float, dist, device=None) -> float:
    """The slowest rank's figure (a time); the value itself without a process group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(world: int, units_per_rank: float, seconds: float) -> float:
    """Whole-job throughput: every rank produced units_per_rank units within the slowest rank's time."""
    return world * units_per_rank / seconds
