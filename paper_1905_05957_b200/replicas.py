"""Multi-GPU form of the step: independent replicas.

The n workers of DoubleSqueeze are rows of one tensor on one GPU, so a second GPU has nothing to
exchange with the first: N GPUs run N independent replicas of the same step.  The only collective
is the one the measurement needs, the maximum over ranks of the timed interval.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(values: list[float], device="cpu") -> list[float]:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(elements_per_replica_step: int, steps: int, slowest_ms: float, world: int) -> float:
    """Whole-job gradient entries per second: every replica did `steps` steps within `slowest_ms`."""
    return world * elements_per_replica_step * steps / (slowest_ms * 1e-3)
