"""Plumbing for multi-process runs (no data-path collective: the hot path does not exchange data)."""
from __future__ import annotations


def max_over_ranks(value: float, device="cpu") -> float:
    """The largest `value` over all ranks of the default process group (the value itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_this_rank: float, device="cpu") -> float:
    """Whole-job throughput in units per second: every rank processed `units_per_rank` units (weak
    scaling), the job took as long as its slowest rank."""
    import torch.distributed as dist
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    return world * units_per_rank / (max_over_ranks(ms_this_rank, device) * 1e-3)
