"""Host-side logic of multi-GPU runs.  The sampling path does not shard across GPUs (a step is a latency chain
that needs the whole state twice); several GPUs run independent replicas -- different streams of the same workload,
one process per GPU, no collective on the data path.  What the ranks share is only the timing protocol: a barrier
on both sides of the timed region, the maximum of the per-rank device times, and the sum of the units produced.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Sequence, Tuple


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


def check_world(asked: int) -> None:
    """The launcher's world size must be the number of replicas asked for: a run that was asked for N GPUs and got another
    number of ranks stops here instead of reporting a figure for a different job."""
    _, world, _ = rank_env()
    if world != asked:
        raise SystemExit("asked for %d replicas but the launcher started %d ranks (WORLD_SIZE); refusing to measure" % (asked, world))


def needs_launch(asked: int) -> bool:
    """True when several replicas were asked for and no launcher has set up the ranks yet."""
    return asked > 1 and "WORLD_SIZE" not in os.environ


def launch_local(n: int, argv: Sequence[str], timeout_s: float = 3600.0) -> int:
    """Start n ranks of `argv` on this node (one process per GPU: RANK = LOCAL_RANK = 0..n-1, rendezvous on 127.0.0.1 at
    a free port), pass rank 0's standard output through and wait for all of them.  Returns 0 when every rank exited 0;
    otherwise the first non-zero exit code, after the remaining ranks have been stopped (only the processes started
    here are touched)."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs: List[subprocess.Popen] = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env, stdout=None if rank == 0 else subprocess.DEVNULL))
    rc = 0
    try:
        for p in procs:
            r = p.wait(timeout=timeout_s)
            if r != 0 and rc == 0:
                rc = r
                break
    except subprocess.TimeoutExpired:
        rc = 124
    if rc != 0:
        for p in procs:
            if p.poll() is None:
                p.kill()
        print("replica launch failed: a rank exited with code %d" % rc, file=sys.stderr)
    return rc
