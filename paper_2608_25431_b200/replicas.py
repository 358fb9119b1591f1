"""Replica bookkeeping for runs on more than one GPU.

The path does not shard: segments are independent and each GPU runs its own replica of
the workload with no data-path collective.  The only communication is for measurement:
a barrier around the timed region and the maximum of the per-rank times, so that the
whole-job throughput is (sum of the replicas' payload) / (slowest rank's time).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world():
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def slowest(ms: float, device="cpu") -> float:
    """Maximum over ranks of a per-rank duration."""
    if world() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def total(x: float, device="cpu") -> float:
    """Sum over ranks (payload bytes, launches)."""
    if world() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(payload_bytes: float, ms: float, device="cpu"):
    """(whole-job GB/s, slowest rank's ms) from this rank's payload and duration."""
    worst = slowest(ms, device)
    return total(payload_bytes, device) / (worst * 1e-3) / 1e9, worst
