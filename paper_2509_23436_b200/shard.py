"""Host-side sharding of the LOT attention forward over ranks.

The (batch, head) slices of a call are independent problems (per-head pivots, no cross-head or
cross-batch term anywhere in Eq. (1)-(4)), so N ranks split them with no data-path collective:
every rank runs the same library call on its own block of slices and owns the matching block of
the output.  The only collectives are the timing barrier and a MAX over the ranks' elapsed times.

A block is a rectangle [b_lo, b_hi) x [h_lo, h_hi) of the (batch, head) grid, so that each rank's
tensors stay dense [B', H', n, d] arrays with their own pivots z[h_lo:h_hi], beta[h_lo:h_hi]:
  * world <= B: the batch rows are dealt out as evenly as possible, all heads each;
  * world  > B and B divides world: every batch row is shared by world / B ranks, which deal out
    its heads (the long-context workload has B = 1, H = 16: N ranks take H / N heads each);
  * otherwise the batch split is used and ranks beyond B get an empty block.
"""
from __future__ import annotations

from typing import Callable, Optional


def batch_block(B: int, world: int, rank: int) -> tuple[int, int]:
    """[lo, hi) of `rank` when B items are split over `world` ranks as evenly as possible."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def slice_block(B: int, H: int, world: int, rank: int) -> tuple[int, int, int, int]:
    """(b_lo, b_hi, h_lo, h_hi): the rectangle of (batch, head) slices `rank` owns."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    if B > 0 and world > B and world % B == 0:
        per_row = world // B
        b = rank // per_row
        h_lo, h_hi = batch_block(H, per_row, rank % per_row)
        return b, b + 1, h_lo, h_hi
    b_lo, b_hi = batch_block(B, world, rank)
    return b_lo, b_hi, 0, H


def shard_inputs(q, k, v, z, beta, key_len, world: int, rank: int):
    """The block of `rank` cut out of full-size inputs (torch tensors or numpy arrays alike).

    Returns (block, q, k, v, z, beta, key_len) with block = slice_block(...).  Cutting heads out of
    a B > 1 tensor gives a strided view; callers that need dense memory make it contiguous.
    """
    B, H = q.shape[0], q.shape[1]
    blk = slice_block(B, H, world, rank)
    b0, b1, h0, h1 = blk
    cut = lambda t: t[b0:b1, h0:h1]
    kl = None if key_len is None else key_len[b0:b1]
    return blk, cut(q), cut(k), cut(v), z[h0:h1], beta[h0:h1], kl


def run_sharded(forward: Callable, q, k, v, z, beta, key_len, world: int, rank: int):
    """Run `forward(q, k, v, z, beta, key_len)` on this rank's block; returns (block, result or None).

    `forward` is the library call on a GPU rank and the CPU checker in the host-only tests: the split
    itself is the same code in both.  A rank whose block is empty calls nothing.
    """
    blk, qs, ks, vs, zs, bs, kl = shard_inputs(q, k, v, z, beta, key_len, world, rank)
    b0, b1, h0, h1 = blk
    if b1 <= b0 or h1 <= h0:
        return blk, None
    return blk, forward(qs, ks, vs, zs, bs, kl)


def job_throughput(units_per_rank: list[int], seconds_per_rank: list[float]) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return sum(units_per_rank) / max(seconds_per_rank)
