"""Replica bookkeeping for multi-GPU runs.

The path has no exchange step: N GPUs run N independent replicas, each generating its own
portfolio.  The only collectives are a barrier around the timed region and the max over ranks of
the elapsed times, from which the whole-job figure is derived.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def ms_per_variant(step_ms_max: float, variants_per_replica: int, world: int) -> float:
    """Whole-job time per variant: every replica finishes `variants_per_replica` variants in a step."""
    return step_ms_max / (variants_per_replica * world)
