"""Multi-rank form of the path on CPU ranks (gloo): one pool split by attention heads.

What is checked: the head shards partition the heads exactly once with GQA groups intact; every rank
running the attention definition (the CPU oracle) on its head slice and the ranks' results put together
equal the unsharded result; dK / dV are summed over the ranks that share a kv head; the measurement
bookkeeping takes the slowest rank and the summed work."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2607_23250_b200 import pools, sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("hq,hkv,world", [(32, 8, 1), (32, 8, 2), (32, 8, 4), (32, 8, 8), (32, 4, 8), (64, 4, 16),
                                          (8, 2, 4), (4, 4, 2), (128, 4, 8)])
def test_head_groups_partition_the_heads(hq, hkv, world):
    G = hq // hkv
    shards = [sharding.head_groups(hq, hkv, world, r) for r in range(world)]
    q_all = sorted(h for s in shards for h in s.q_heads)
    assert q_all == list(range(hq))                                    # every query head exactly once
    for s in shards:
        assert all(h // G in s.kv_heads for h in s.q_heads)            # a query head sits with its kv head
        assert len(s.q_heads) == hq // world
        # the slice is group-contiguous: local query head i reads local kv head i // (local G)
        g_local = s.hq // s.hkv
        for i, h in enumerate(s.q_heads):
            assert s.kv_heads[i // g_local] == h // G
        assert s.rank in s.kv_sharers
        for other in s.kv_sharers:
            assert shards[other].kv_heads == s.kv_heads
    if world <= hkv:
        assert sorted(h for s in shards for h in s.kv_heads) == list(range(hkv))    # kv heads exactly once
        assert all(len(s.kv_sharers) == 1 for s in shards)
    else:
        assert all(len(s.kv_sharers) == world // hkv and s.hkv == 1 for s in shards)


def test_head_groups_reject_impossible_splits():
    for hq, hkv, world in [(32, 8, 3), (32, 8, 64), (8, 2, 3), (8, 3, 2)]:
        with pytest.raises(ValueError):
            sharding.head_groups(hq, hkv, world, 0)


def _worker(rank, world, port, hq, hkv, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lengths = [70, 1, 130, 55]
    d = 16
    cu = pools.cu_seqlens(lengths)
    T = int(cu[-1])
    t = pools.make_tensors(T, hq, hkv, d, seed=5)                       # the same pool on every rank
    shard = sharding.head_groups(hq, hkv, world, rank)
    groups = sharding.kv_subgroups(hq, hkv, world)
    q, k, v, dout = sharding.slice_heads(shard, t["q"], t["k"], t["v"], t["dout"])
    f = lambda x: x.float().numpy()
    o, lse = oracle.attn_fwd(f(q), f(k), f(v), cu)
    dq, dk, dv = oracle.attn_bwd(f(q), f(k), f(v), o, lse, f(dout), cu)
    dk_t, dv_t = sharding.reduce_kv_grads(shard, torch.from_numpy(dk), torch.from_numpy(dv),
                                          group=groups.get(shard.kv_heads[0]))
    work = float(len(shard.q_heads))
    ms, total = sharding.aggregate(10.0 + rank, work)
    out[rank] = dict(shard=shard, o=o, lse=lse, dq=dq, dk=dk_t.numpy(), dv=dv_t.numpy(), ms=ms, total=total)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("hq,hkv,world", [(4, 2, 2), (8, 2, 4)], ids=["kv_heads_split", "kv_head_shared"])
def test_ranks_reproduce_the_unsharded_result(hq, hkv, world):
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), hq, hkv, out), nprocs=world, join=True)
    assert set(out.keys()) == set(range(world))
    lengths = [70, 1, 130, 55]
    cu = pools.cu_seqlens(lengths)
    t = pools.make_tensors(int(cu[-1]), hq, hkv, 16, seed=5)
    f = {n: x.float().numpy() for n, x in t.items()}
    o, lse = oracle.attn_fwd(f["q"], f["k"], f["v"], cu)
    dq, dk, dv = oracle.attn_bwd(f["q"], f["k"], f["v"], o, lse, f["dout"], cu)
    for r in range(world):
        res = out[r]
        s = res["shard"]
        qh, kh = list(s.q_heads), list(s.kv_heads)
        # heads are independent: a rank's outputs are the unsharded ones, bit for bit
        assert np.array_equal(res["o"], o[:, qh]) and np.array_equal(res["lse"], lse[qh])
        assert np.array_equal(res["dq"], dq[:, qh])
        if len(s.kv_sharers) == 1:
            assert np.array_equal(res["dk"], dk[:, kh]) and np.array_equal(res["dv"], dv[:, kh])
        else:                                   # partial sums over query heads, added across the sub-group
            assert np.abs(res["dk"] - dk[:, kh]).max() <= 1e-5 * np.abs(dk).max()
            assert np.abs(res["dv"] - dv[:, kh]).max() <= 1e-5 * np.abs(dv).max()
        assert res["ms"] == 10.0 + world - 1     # the slowest rank decides
        assert res["total"] == float(hq)         # work adds up to the whole pool's heads
    assert sharding.aggregate(3.0, 5.0) == (3.0, 5.0)          # single-process path is the identity


def test_rank_spec_is_one_pool_or_replicas():
    assert sharding.rank_spec(2, 0.0, 3).seed == 0                       # head-sharded: the same pool everywhere
    assert sharding.rank_spec(2, 0.0, 3, replicas=True).seed == 3        # replicas: one pool per rank
    assert sharding.rank_spec(2, 0.0, 0, n_seqs=1).total_tokens == 32768
