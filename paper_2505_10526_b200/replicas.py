"""Multi-GPU arrangement of the verify step: independent replicas.

Sequences do not interact and every GPU holds the whole LM head, so the path
has no exchange step.  N GPUs run N replicas of the step, one process per GPU;
the only communication is the barrier around the timed region and the
max-over-ranks of the per-step time.  These helpers hold that host-side logic so
that it can be exercised on CPU with the gloo backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_size() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's value (every rank receives it)."""
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: int, ms_local: float, device="cpu"):
    """Whole-job throughput of N replicas: all ranks' units over the slowest rank's time.
    Returns (ms_per_step, units_per_second)."""
    ms = max_over_ranks(ms_local, device)
    return ms, world_size() * units_per_rank / (ms * 1e-3)


def barrier() -> None:
    if world_size() > 1:
        dist.barrier()
