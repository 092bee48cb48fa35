"""Host-side helpers for running the path on several GPUs of one node.

The linear layer's output rows (tokens) are independent of one another (each
row of Y depends on one row of X and on the whole weight), so the path shards
by tokens: every rank holds the packed weights and works on its own rows with
no collective on the data path.  A per-tensor activation scale computed from
the data would need one scalar max across ranks; a sharded deployment supplies
the scale instead (GPUSQ_SCALE_GIVEN).  The only communication is the timing
reduction of the benchmark.  No arithmetic of the method lives here.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_rows(M: int, world: int, rank: int) -> Tuple[int, int]:
    """Rows [lo, hi) of an [M, K] activation tensor that `rank` of `world` works on.

    Contiguous, non-overlapping, covering 0..M; sizes differ by at most one row.
    """
    if world <= 0 or not 0 <= rank < world:
        raise ValueError("rank %d outside world %d" % (rank, world))
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device: torch.device) -> float:
    """The largest `value` over all ranks (the time of the slowest rank); the value itself without a group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: float, seconds_slowest_rank: float, world: int) -> float:
    """Units all ranks processed per second of the slowest rank (weak scaling: every rank does `units_per_rank`)."""
    return world * units_per_rank / seconds_slowest_rank
