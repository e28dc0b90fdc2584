"""Host-side plumbing of a multi-GPU run: one process per GPU, every rank an independent batch.

The hot path partitions by batch (or by KV-head group) and has no exchange step, so there is no
data-path collective: ranks only meet in a barrier and in the reduction of their timings.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import synth


def rank_workload(name: str, seed: int, rank: int, world: int, max_heads: int = 0) -> synth.Workload:
    """The batch of one rank: same workload recipe on every rank, seed offset by the rank."""
    w = synth.make_workload(name, seed=seed + (rank if world > 1 else 0))
    if max_heads > 0:
        w = synth.reduced(w, len_div=1, max_heads=max_heads)
    return w


def aggregate(ms: float, flops: float, device) -> tuple[float, float]:
    """Whole-job figures from per-rank ones: (max over ranks of the elapsed ms, sum of the FLOPs)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), float(flops)
    t_max = torch.tensor([ms], dtype=torch.float64, device=device)
    t_sum = torch.tensor([flops], dtype=torch.float64, device=device)
    dist.all_reduce(t_max, op=dist.ReduceOp.MAX)
    dist.all_reduce(t_sum, op=dist.ReduceOp.SUM)
    return float(t_max[0]), float(t_sum[0])


def throughput_tflops(ms_total: float, steps: int, flops_total: float) -> float:
    """Whole-job TFLOPS: the FLOPs all ranks processed per step over the slowest rank's step time."""
    return flops_total / (ms_total / steps * 1e-3) / 1e12
