"""Plumbing for running one replica per GPU: positions are independent, so ranks
share nothing on the data path; only the timing is reduced across ranks."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the torchrun environment; (0, 1, 0) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: torch.device | None = None) -> bool:
    """Join the process group when WORLD_SIZE > 1.  Returns True if a group was created."""
    rank, world, _ = env_rank_world()
    if world <= 1:
        return False
    kwargs = {}
    if backend == "nccl" and device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return True


def max_over_ranks(value: float, device: torch.device) -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def whole_job_rate(units_per_rank: int, steps: int, world: int, elapsed_ms_max: float) -> float:
    """Units per second of the whole job: every rank processed units_per_rank * steps units
    in the time the slowest rank took."""
    return units_per_rank * world * steps / (elapsed_ms_max * 1e-3)


def shard_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own batch of positions."""
    return base_seed + rank


def finalize() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
