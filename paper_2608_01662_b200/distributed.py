"""Multi-rank plumbing of the benchmark: one process per GPU, independent units per rank, no data-path collective.

The path shards by independent units (query chunks of a prefill, sequences of a decode batch), so each rank runs
its own units and the ranks only meet to agree on the time: the slowest rank's device time bounds the job.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(value: float, device="cpu") -> float:
    """The maximum of `value` over all ranks (the value itself when there is one process)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world: int, ms_per_step_max: float) -> float:
    """Whole-job units per second: every rank processed units_per_rank units in the slowest rank's time."""
    return units_per_rank * world / (ms_per_step_max * 1e-3)


def shard_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous share of n_units independent units for `rank` (sizes differ by at most one)."""
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))
