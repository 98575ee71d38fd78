"""Replica bookkeeping for multi-GPU runs.

The hot path has no exchange step: every (batch entry, layer, key head) is independent, so N GPUs
run N independent replicas of the workload.  The only cross-rank arithmetic is the benchmark's:
the job's time is the slowest rank's, the job's work is the sum over ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def job_time_and_work(local_ms: float, local_units: float, device="cpu", group=None):
    """Returns (max over ranks of local_ms, sum over ranks of local_units).  Works without an
    initialised process group (single replica)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(local_ms), float(local_units)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(u, op=dist.ReduceOp.SUM, group=group)
    return float(t.item()), float(u.item())


def job_throughput(local_ms: float, local_units: float, device="cpu", group=None) -> float:
    """Whole-job units per second: all ranks' units / slowest rank's time."""
    ms, units = job_time_and_work(local_ms, local_units, device, group)
    return units / (ms * 1e-3)
