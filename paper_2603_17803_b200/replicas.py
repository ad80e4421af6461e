"""Multi-process plumbing for running independent replicas of the path, one process per GPU.

The path has no exchange step on one GPU and is specified as single-GPU, so ranks never exchange data:
the process group is used for the timing barrier and for the max-over-ranks reduction of the measured time.
"""
from __future__ import annotations

import os
from typing import Sequence

import torch
import torch.distributed as dist


def env_world():
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> None:
    world, _, _ = env_world()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def replica_seed(rank: int, data_set: int) -> int:
    """Every rank draws its own data sets (weak scaling: fixed work per GPU)."""
    return 1000 * rank + data_set


def aggregate_steps_per_s(world: int, steps: int, max_ms: float) -> float:
    """Whole-job throughput: every rank ran `steps` steps, the job took the slowest rank's time."""
    return world * steps / (max_ms / 1e3)


def shutdown() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
