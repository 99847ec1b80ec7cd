"""Aggregation of per-rank timings when N independent replicas run, one process per GPU.

The encrypted linear layer does not shard across GPUs (nothing in the method exchanges data), so a
multi-GPU run is N replicas, each decoding its own token stream.  The only communication is the
reduction of the timing itself: the job's step time is the slowest rank's, and the job-level latency
per token is that time divided by the number of streams decoded in parallel.
"""
from __future__ import annotations


def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's time; a no-op without an initialised process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_ms_per_token(ms_per_step_max: float, world_size: int) -> float:
    """Whole-job latency per decoded token with world_size independent streams."""
    return ms_per_step_max / max(1, world_size)
