"""Rank plumbing for running independent replicas of the block on several GPUs.

The SPA block has no exchange step (images are independent), so N GPUs run N replicas of the same
per-GPU work; the only cross-rank operations are a barrier and the reductions that turn per-rank
measurements into one whole-job figure.  The helpers work with any torch.distributed backend (NCCL on
GPUs, gloo on CPU for tests) and degrade to no-ops in a single process.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world() -> tuple:
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device=None) -> int:
    """Join the process group when launched with more than one rank; returns the world size."""
    _, _, n = world()
    if n > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, **kw)
    return n


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def reduce_scalar(value: float, op: str, device="cpu") -> float:
    """max or sum of a per-rank scalar over all ranks (the value itself in a single process)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_local: float, ms_local: float, device="cpu") -> tuple:
    """Whole-job throughput of independent replicas: all units processed by all ranks divided by the
    slowest rank's time.  Returns (units per second, max time in ms)."""
    ms = reduce_scalar(ms_local, "max", device)
    units = reduce_scalar(units_local, "sum", device)
    return units / (ms * 1e-3), ms


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
