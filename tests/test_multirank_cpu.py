"""The N>1 path on CPU: gloo ranks split the (batch, head) slices of one call through shard.run_sharded, the same
function bench.py drives on GPU ranks; each computes its block with no data exchange, and the gathered blocks
equal the unsharded result (the slices are independent).  The float64 CPU oracle stands in for the device call
here: what is tested is the host-side split (by batch rows, and by heads when there are more ranks than rows),
the gather and the max-over-ranks timing reduction."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import lot_oracle as O
from paper_2509_23436_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle_forward(x):
    def fwd(q, k, v, z, beta, key_len):
        return O.attention_fwd(np.ascontiguousarray(q), np.ascontiguousarray(k), np.ascontiguousarray(v), z, beta,
                               x.eps, x.iters, key_len=key_len)
    return fwd


def _worker(rank, world, port, ret, B, H):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = synth.make(B, H, 40, 16, 4, seed=17, eps=0.2, iters=5, key_len_range=(20, 40))
    d = x.f64()
    blk, mine = shard.run_sharded(_oracle_forward(x), d["q"], d["k"], d["v"], d["z"], d["beta"], d["key_len"], world, rank)
    blocks = [None] * world
    dist.all_gather_object(blocks, (blk, mine))
    t = torch.tensor([0.5 + rank], dtype=torch.float64)          # pretend elapsed seconds
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        full = np.full_like(d["q"], np.nan)
        for (b0, b1, h0, h1), part in blocks:
            if part is not None:
                full[b0:b1, h0:h1] = part
        ref = O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters, key_len=d["key_len"])
        ret["err"] = float(np.abs(full - ref).max())
        ret["tmax"] = float(t.item())
        ret["cover"] = sorted(b[0] for b in blocks)
    dist.destroy_process_group()


def _run(world, B, H):
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), ret, B, H), nprocs=world, join=True)
        return dict(ret)


def test_two_ranks_split_the_batch_without_exchange():
    ret = _run(2, 3, 2)
    assert ret["err"] == 0.0
    assert ret["tmax"] == 1.5
    assert ret["cover"] == [(0, 2, 0, 2), (2, 3, 0, 2)]


def test_two_ranks_split_the_heads_of_a_single_batch_row():
    """The long-context workload has one batch row: the ranks deal out its heads, each with its own pivots."""
    ret = _run(2, 1, 5)
    assert ret["err"] == 0.0
    assert ret["cover"] == [(0, 1, 0, 3), (0, 1, 3, 5)]


def test_slice_block_covers_the_grid_exactly_once():
    for B, H, world in ((1, 16, 8), (1, 16, 3), (2, 6, 4), (2, 6, 8), (5, 3, 2), (3, 4, 7), (4, 8, 1)):
        seen = np.zeros((B, H), dtype=int)
        for r in range(world):
            b0, b1, h0, h1 = shard.slice_block(B, H, world, r)
            seen[b0:b1, h0:h1] += 1
        assert (seen == 1).all(), (B, H, world)


def test_batch_block_partitions_and_throughput():
    for B in (0, 1, 5, 8, 17):
        for world in (1, 2, 3, 8):
            blocks = [shard.batch_block(B, world, r) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(blocks, blocks[1:]))
            sizes = [hi - lo for lo, hi in blocks]
            assert max(sizes) - min(sizes) <= 1
    assert shard.job_throughput([100, 100], [1.0, 2.0]) == 100.0
