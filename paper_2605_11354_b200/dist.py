"""Process-group plumbing for multi-GPU benchmark runs.

The SLA forward has no exchange step: every (batch, head) problem is independent, so several GPUs run
independent replicas of the workload and no collective touches the data path.  torch.distributed is used
only to line the ranks up (barrier) and to take the maximum of their device-measured times.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when run directly."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(backend: str | None = None):
    """Join the process group if a launcher started more than one rank; returns (rank, local_rank, world)."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        kwargs = {}
        if backend == "nccl":
            kwargs["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return rank, local_rank, world


def barrier(device=None):
    if dist.is_initialized():
        if device is not None and device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def max_over_ranks(value: float, device=None) -> float:
    """Largest of the per-rank values (each rank passes its own device-measured time)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, local_seconds: float, device=None) -> tuple[float, float]:
    """Whole-job throughput of independent replicas: all ranks' units over the slowest rank's time.
    Returns (units_per_second, max_seconds)."""
    worst = max_over_ranks(local_seconds, device)
    total = sum_over_ranks(units_per_rank, device)
    return total / worst, worst


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
