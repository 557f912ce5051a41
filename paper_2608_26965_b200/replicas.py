"""Plumbing for running independent replicas of the hot path on several GPUs.

Heads (and batch items) are independent through every stage, so nothing on the
data path is exchanged between ranks: each rank runs its own replica and the
ranks only meet at a barrier and to agree on the slowest rank's time.  The
same functions run over `gloo` on CPU (tests) and over `nccl` on GPUs (bench).
"""
from __future__ import annotations

import os
from typing import Optional

import torch
import torch.distributed as dist


def world() -> tuple:
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device: Optional[torch.device] = None) -> bool:
    """Joins the process group when launched with more than one rank."""
    _, _, size = world()
    if size <= 1:
        return False
    if not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return True


def barrier(device: Optional[torch.device] = None) -> None:
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)
    if dist.is_initialized():
        dist.barrier()
        if device is not None and device.type == "cuda":
            torch.cuda.synchronize(device)


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """The slowest rank's time (what a weak-scaling throughput must be divided by)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or torch.device("cpu"))
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_this_rank: float, device: Optional[torch.device] = None) -> dict:
    """Whole-job throughput of N replicas: all ranks' units over the slowest rank's time."""
    _, _, size = world()
    ms = max_over_ranks(ms_this_rank, device)
    return {"ms": ms, "value": size * units_per_rank / (ms * 1e-3), "n": size}


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
