"""Replica bookkeeping for multi-GPU runs.

The path never exchanges data between GPUs (each rank moves its own KV over its own
host link), so N GPUs are N independent replicas.  The only cross-rank arithmetic is
the reporting rule: the job's time is the slowest rank's time and the job's work is
the sum of every rank's work.  It is kept here, away from CUDA, so it can be tested
with the gloo backend on CPU.
"""
from __future__ import annotations

from typing import Tuple


def job_totals(ms_per_step: float, units_per_step: float, dist=None, device=None) -> Tuple[float, float]:
    """(max over ranks of ms_per_step, sum over ranks of units_per_step).
    `dist` is torch.distributed when a process group is up, else None (one replica)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms_per_step, units_per_step
    import torch
    t = torch.tensor([ms_per_step], dtype=torch.float64, device=device)
    u = torch.tensor([units_per_step], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
