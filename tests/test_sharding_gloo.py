"""World-size-2 check of the multi-GPU bookkeeping on CPU (gloo): every rank gets its own pool and
the aggregate is (slowest rank, summed work)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_23250_b200 import pools, sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = sharding.rank_spec(2, 0.0, rank, n_seqs=1)
    lengths = pools.pool_lengths(spec)
    work = float(sum(l * (l + 1) // 2 for l in lengths))
    ms, total = sharding.aggregate(10.0 + rank, work)
    out[rank] = (ms, total, work, len(lengths), sum(lengths))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_get_distinct_pools_and_aggregate():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    (ms0, tot0, w0, n0, t0), (ms1, tot1, w1, n1, t1) = out[0], out[1]
    assert ms0 == ms1 == 11.0                      # the slowest rank decides
    assert tot0 == tot1 == w0 + w1                 # work adds up
    assert t0 == t1 == 32768 and w0 != w1          # same shape, different samples
    # single-process path is the identity
    assert sharding.aggregate(3.0, 5.0) == (3.0, 5.0)
    assert sharding.rank_spec(2, 0.0, 0).seed == 0 and sharding.rank_spec(2, 0.0, 3).seed == 3
