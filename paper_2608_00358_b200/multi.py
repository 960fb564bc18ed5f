"""Replica bookkeeping for runs on more than one GPU.

The path has no exchange between GPUs (every rank of a collective is virtual and lives in one GPU's memory),
so N GPUs run N independent replicas. The only cross-process steps are a barrier around the timed region and
the max over ranks of the region's duration; the whole-job figure is the bytes all replicas moved over that
maximum. `torch.distributed` is used for exactly that (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Optional

import torch


def replica_throughput_gbs(local_ms: float, bytes_per_step: int, steps: int, dist=None, device: Optional[str] = None):
    """Returns (whole-job GB/s, max-over-ranks milliseconds for the `steps` steps). Every rank gets the same
    answer. With dist None (a single process) it is just this process's own figure."""
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device or "cpu")
    world = 1
    if dist is not None and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        world = dist.get_world_size()
    worst_ms = float(t.item())
    return world * bytes_per_step * steps / (worst_ms * 1e-3) / 1e9, worst_ms


def barrier(dist=None):
    if dist is not None and dist.is_initialized():
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()
