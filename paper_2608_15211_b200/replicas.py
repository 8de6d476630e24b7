"""Replicas-only multi-GPU accounting.

Nothing of the attention block is sharded and there is no collective on the data path: with N GPUs the
benchmark runs N independent replicas of the same workload.  The only exchange is the timing reduction: the
step time of the job is the slowest replica's, and the job's throughput is N times one replica's work over
that time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(ms: float, device: str = "cpu") -> float:
    """The largest `ms` over all ranks (the value itself without an initialised process group)."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flop_per_replica: float, world: int, ms_per_step: float) -> float:
    """Aggregate TFLOP/s of `world` replicas that each do `flop_per_replica` in `ms_per_step`."""
    return world * flop_per_replica / (ms_per_step * 1e-3) / 1e12
