"""Aggregation of per-rank timings for independent replicas (one process per GPU).

The NVFP4 linear path has no exchange step, so N GPUs run N independent replicas; the only
communication is for timing: a barrier around the timed region, the maximum step time over
ranks, and the sum of the work all ranks did.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def aggregate(ms_local: float, units_local: float, device="cpu"):
    """Returns (max milliseconds over ranks, total units over ranks, world size)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(ms_local), float(units_local), 1
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item()), dist.get_world_size()


def throughput(ms_local: float, units_local: float, device="cpu") -> float:
    """Whole-job units per second: total units of all ranks / slowest rank's time."""
    ms, units, _ = aggregate(ms_local, units_local, device)
    return units / (ms * 1e-3)
