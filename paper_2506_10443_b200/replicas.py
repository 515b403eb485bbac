"""Multi-GPU form of the workload: independent replicas.

The linear layer has no exchange step (rows of W are independent and the benchmark does not shard
a single matrix), so N GPUs run N copies of the same step and nothing crosses NVLink on the data
path.  The only collective is the timing reduction: a step's time is the MAXIMUM over the ranks,
and the job's throughput is the units all ranks processed divided by that time.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def max_over_ranks(values: Sequence[float], device: str = "cpu") -> list:
    """Element-wise maximum of ``values`` over all ranks of the default process group (the values
    themselves when no group is initialised).  Works with gloo (CPU tensors) and nccl (CUDA)."""
    if not (dist.is_available() and dist.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def aggregate_throughput(units_per_rank_step: float, steps: int, elapsed_ms_this_rank: float, world: int,
                         device: str = "cpu") -> dict:
    """Whole-job throughput of ``world`` replicas: units of all ranks / max-over-ranks time."""
    (ms,) = max_over_ranks([elapsed_ms_this_rank], device)
    per_s = units_per_rank_step * steps * world / (ms * 1e-3)
    return {"ms": ms, "ms_per_step": ms / steps, "units_per_s": per_s, "units_per_s_one_replica": per_s / world}
