"""Multi-GPU plumbing of the benchmark: the path does not shard ("replicas only"), so N GPUs
run N independent replicas; the only cross-rank steps are a barrier around the timed region
and a MAX over ranks of the measured times.  Works with any torch.distributed backend (NCCL on
GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Sequence


def max_over_ranks(values: Sequence[float], device=None):
    """Element-wise maximum of `values` over all ranks (identity when not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_throughput(units_per_rank_per_step: int, steps: int, ms_total_this_rank: float, device=None):
    """Whole-job throughput: units all ranks processed / slowest rank's time.  Returns
    (units_per_second, ms_total_max)."""
    import torch.distributed as dist
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    ms = max_over_ranks([ms_total_this_rank], device)[0]
    return world * units_per_rank_per_step * steps / (ms * 1e-3), ms
