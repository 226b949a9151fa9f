"""The N>1 path on CPU: two gloo ranks split the batch of one call, each computes its block with no
data exchange, and the gathered blocks equal the unsharded result (the slices are independent).
The float64 CPU oracle stands in for the device call here: what is tested is the host-side split,
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


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = synth.make(3, 2, 40, 16, 4, seed=17, eps=0.2, iters=5, key_len_range=(20, 40))
    d = x.f64()
    lo, hi = shard.batch_block(3, world, rank)
    mine = O.attention_fwd(d["q"][lo:hi], d["k"][lo:hi], d["v"][lo:hi], d["z"], d["beta"], x.eps, x.iters,
                           key_len=d["key_len"][lo:hi])
    blocks = [None] * world
    dist.all_gather_object(blocks, (lo, hi, mine))
    t = torch.tensor([0.5 + rank], dtype=torch.float64)          # pretend elapsed seconds
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        full = np.concatenate([b[2] for b in sorted(blocks, key=lambda b: b[0])], axis=0)
        ref = O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters, key_len=d["key_len"])
        ret["err"] = float(np.abs(full - ref).max())
        ret["tmax"] = float(t.item())
        ret["cover"] = sorted((b[0], b[1]) for b in blocks)
    dist.destroy_process_group()


def test_two_ranks_split_the_batch_without_exchange():
    world = 2
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
        assert ret["err"] == 0.0
        assert ret["tmax"] == 1.5
        assert ret["cover"] == [(0, 2), (2, 3)]


def test_batch_block_partitions_and_throughput():
    for B in (0, 1, 5, 8, 17):
        for world in (1, 2, 3, 8):
            blocks = [shard.batch_block(B, world, r) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(blocks, blocks[1:]))
            sizes = [hi - lo for lo, hi in blocks]
            assert max(sizes) - min(sizes) <= 1
    assert shard.job_throughput([100, 100], [1.0, 2.0]) == 100.0
