"""Replica bookkeeping for multi-GPU runs.

The verifier path does not shard: with N GPUs, N independent replicas each verify their own
GEMMs (one process per GPU, no data-path collective).  The only cross-rank steps are a barrier
around the timed region and taking the slowest rank's time; they live here so that they can be
exercised with the gloo backend on CPU.
"""
from __future__ import annotations

from typing import Sequence

import torch


def max_over_ranks(values: Sequence[float], dist=None, device="cpu") -> list:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_throughput(units_per_rank: float, seconds_slowest: float, world_size: int) -> float:
    """Weak scaling: every rank processes `units_per_rank` in the time of the slowest rank."""
    return units_per_rank * world_size / seconds_slowest
