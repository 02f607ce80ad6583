"""Host-side plumbing for running independent replicas of the hot path on several GPUs.

Requests are independent and the path has no exchange step, so multi-GPU operation means one process
per GPU, each running its own batch (no collective on the data path).  The only communication is for
measurement: a barrier around the timed region and a MAX reduction of the per-rank device time."""
from __future__ import annotations

import os
from typing import Optional

import torch
import torch.distributed as dist


def env_rank_world():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))


def init_replicas(backend: str, device: Optional[torch.device] = None) -> None:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (no-op at world size 1)."""
    rank, world, _ = env_rank_world()
    if world <= 1 or dist.is_initialized():
        return
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = device
    dist.init_process_group(backend, rank=rank, world_size=world, **kw)


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own batch: seeds of different ranks never collide with the per-round seeds."""
    return base_seed + 17 * rank


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: torch.device) -> float:
    """MAX over ranks of a scalar (the slowest rank's time decides the whole job's time)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rounds_per_second(steps_per_rank: int, world: int, max_ms: float) -> float:
    """Rounds completed by all ranks together per second of the slowest rank."""
    return world * steps_per_rank / (max_ms * 1e-3)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
