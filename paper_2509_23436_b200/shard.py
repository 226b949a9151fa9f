"""Host-side sharding of the LOT attention forward over ranks.

The (batch, head) slices of a call are independent problems (per-head pivots, no cross-head or
cross-batch term anywhere in Eq. (1)-(4)), so N ranks split the batch with no data-path
collective: rank k takes a contiguous block of batch rows, runs the same call on it, and owns the
matching rows of the output.  The only collectives are the timing barrier and a MAX over the
ranks' elapsed times.
"""
from __future__ import annotations


def batch_block(B: int, world: int, rank: int) -> tuple[int, int]:
    """[lo, hi) batch rows of `rank` when B rows are split over `world` ranks as evenly as possible."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def job_throughput(units_per_rank: list[int], seconds_per_rank: list[float]) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return sum(units_per_rank) / max(seconds_per_rank)
