"""Multi-GPU plumbing of the benchmark: replicas only.

The per-layer decode step of one token stream does not shard: its K experts are already spread over
all SMs of one GPU and the step is latency-bound, so a second GPU can only serve another stream.
N ranks are therefore N independent replicas, each with its own layer instances and its own
routing; there is no data-path collective.  The only communication is the timing protocol: a
barrier before the timed region and a MAX over the ranks' device times after it.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def first_instance(rank: int, instances_per_rank: int) -> int:
    """Rank r serves layer instances [r * n, (r + 1) * n): seeded independently, disjoint."""
    return rank * instances_per_rank


def max_over_ranks(ms: float, device: torch.device | str = "cpu") -> float:
    """Slowest rank's time for the same timed region (the job is over when the last rank is)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, units_per_rank: int, ms_max: float) -> float:
    """Units per second over all ranks: every rank did `units_per_rank` within `ms_max`."""
    return world * units_per_rank / (ms_max * 1e-3)
