"""Host-side plumbing for running independent replicas of the step on several GPUs of one node.

The hot path has no exchange step (token rows are independent and every GPU holds the full packed
weight), so there is no data-path collective: ranks only agree on the slowest rank's time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(value: float, device=None) -> float:
    """The maximum of a per-rank scalar (e.g. elapsed milliseconds) over all ranks."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: float, steps: int, max_ms: float, world: int) -> float:
    """Units processed by all ranks divided by the slowest rank's time (units per second)."""
    return world * units_per_rank_per_step * steps / (max_ms * 1e-3)
