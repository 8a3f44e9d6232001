"""Replica-only scaling: one request at batch size one does not shard (a layer-by-layer dependent chain), so N GPUs run N
independent handles on N independent requests.  The only cross-rank steps are the barrier around the timed region and
the reduction of the timing; this module holds that host logic so that it can be exercised without GPUs."""
from __future__ import annotations

from typing import Optional

import torch


def max_over_ranks_ms(ms: float, dist=None, device: Optional[torch.device] = None) -> float:
    """The slowest rank's time for the same timed region (all ranks get the same value)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank` within the slowest rank's `ms`."""
    return units_per_rank * world / (ms / 1000.0)


def prints_result(rank: int) -> bool:
    """Only rank 0 prints the result line (and, for the CPU reference arm, only rank 0 runs at all)."""
    return rank == 0
