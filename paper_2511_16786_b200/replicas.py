"""Bookkeeping for running N independent replicas of the compression pass, one process per GPU.

The path needs no exchange between GPUs (every (layer, sequence, head) is independent and the
only cross-layer coupling, the energy sums, stays inside one replica), so the ranks only meet at
a barrier around the timed region and in one MAX reduction of the elapsed time.  Works with the
"nccl" backend on GPUs and with "gloo" on CPU (used by the tests).
"""
from __future__ import annotations

import os

import torch


def world_from_env():
    """(rank, world_size, local_rank) as torch.distributed.run exports them; (0, 1, 0) without it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Joins the process group when WORLD_SIZE > 1; returns the torch.distributed module or None."""
    rank, world, _ = world_from_env()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return dist


def barrier(dist, device=None):
    if dist is not None:
        dist.barrier()
    if device is not None and torch.device(device).type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The slowest rank's time: every multi-GPU number is reported against it."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_replica: float, world: int, ms_per_step: float) -> float:
    """Units all replicas processed per second (weak scaling: per-GPU work is fixed)."""
    return units_per_replica * world / (ms_per_step / 1000.0)
