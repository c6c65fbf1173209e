"""Running N independent replicas of the path, one process per GPU.

The path has no exchange step (channels and sequences are independent, and everything the library does stays on
one device), so several GPUs simply run several copies: each rank draws its own seeded inputs, the ranks meet at a
barrier on both sides of the timed region, the slowest rank's time is the job's time, and the job's throughput is
the work of all ranks over that time.  This module is that bookkeeping; it contains no arithmetic of the method.
"""

from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) for a plain launch."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str, device=None) -> Tuple[int, int]:
    """Join the process group when there is more than one rank.  Returns (rank, world_size)."""
    rank, _, world = env_ranks()
    if world > 1 and not dist.is_initialized():
        if device is not None and backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
    return rank, world


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's figure: what a timed region of the whole job lasted."""
    if world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica works on its own inputs."""
    return int(base_seed) + int(rank)


def whole_job_throughput(units_per_rank: float, ms_slowest: float, world: int) -> float:
    """Units all ranks processed per second, given the slowest rank's time per step (weak scaling)."""
    return world * units_per_rank / (ms_slowest * 1e-3)


def finish(world: int) -> None:
    if world > 1 and dist.is_initialized():
        dist.destroy_process_group()
