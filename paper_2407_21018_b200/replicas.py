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


def torchrun_command(n: int, script: str, script_args, port: int = 0):
    """Command line that starts `n` ranks of `script` on this node, one per GPU, rendezvous on 127.0.0.1."""
    import random
    import sys
    port = port or random.randint(20000, 45000)
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), script] + list(script_args)


def launch(n: int, script: str, script_args, port: int = 0, env=None) -> int:
    """Runs `script` as `n` ranks (see torchrun_command) and returns the launcher's exit code; the ranks'
    output goes to this process's stdout/stderr.  Used when a single-process command line asks for more
    than one replica."""
    import subprocess
    return subprocess.call(torchrun_command(n, script, script_args, port), env=env)
