"""Executing an exchange schedule on CPU ranks (gloo, world size 4): every worker holds its token run of one
pool, sends and receives exactly what the schedule lists, chunk by chunk with the next chunk's receives posted
before the current chunk's compute, runs the attention definition (the CPU oracle) on the tiles placed on it,
and the workers' outputs and gradients put together are the single-pool result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from oracle import schedule as osched
from paper_2607_23250_b200 import exchange, pools

CU = [0, 13, 14, 40, 64]             # samples crossing run and sequence-internal boundaries; ends at a sequence end
SEQ_OFF = [0, 32, 64]                # P = 2 packed sequences x 32 tokens
CP, BLOCK, H, HQ, HKV, D = 2, 8, 2, 8, 2, 8


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _attn_fwd(qf, k, v, a):
    """Rows at sample positions a .. of a sample whose keys 0 .. a + rows are given, by the oracle on the whole prefix."""
    n = k.shape[0]
    full = np.zeros((n, qf.shape[1], qf.shape[2]), np.float32)
    full[a:] = qf.numpy()
    o, lse = oracle.attn_fwd(full, k.numpy(), v.numpy(), [0, n])
    return torch.from_numpy(o[a:]), torch.from_numpy(lse[:, a:])


def _attn_bwd(qf, k, v, o, lse, do, a):
    n = k.shape[0]
    shape = (n, qf.shape[1], qf.shape[2])
    fq, fo, fdo = np.zeros(shape, np.float32), np.zeros(shape, np.float32), np.zeros(shape, np.float32)
    fl = np.zeros((qf.shape[1], n), np.float32)
    fq[a:], fo[a:], fdo[a:], fl[:, a:] = qf.numpy(), o.numpy(), do.numpy(), lse.numpy()
    dq, dk, dv = oracle.attn_bwd(fq, k.numpy(), v.numpy(), fo, fl, fdo, [0, n])     # rows before a have dO = 0: no effect
    return torch.from_numpy(dq[a:]), torch.from_numpy(dk), torch.from_numpy(dv)


def _tensors():
    t = pools.make_tensors(CU[-1], HQ, HKV, D, seed=9)
    return {n: x.float() for n, x in t.items()}          # bf16 values widened: every rank and the check see the same bits


def _worker(rank, world, port, sigma, n_chunks, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lay = exchange.PoolLayout(tuple(CU), tuple(SEQ_OFF), CP, BLOCK, H, HQ, HKV, D)
    rec = osched.schedule(CU, SEQ_OFF, CP, BLOCK, H, sigma)
    t0, t1 = lay.run(rank)
    full = _tensors()
    local = {n: x[t0:t1].contiguous() for n, x in full.items()}          # a worker sees only its own rows
    w = exchange.Worker(rank, lay, sigma, rec, n_chunks, local, _attn_fwd, _attn_bwd, dist, torch)
    o, lse = w.forward()
    dq, dk, dv = w.backward()
    out[rank] = dict(rows=(t0, t1), o=o.numpy(), lse=lse.numpy(), dq=dq.numpy(), dk=dk.numpy(), dv=dv.numpy())
    dist.barrier()
    dist.destroy_process_group()


def _sigmas():
    lay = oracle.tap_layout(CU, SEQ_OFF, CP, BLOCK, H, HQ, HKV, D)
    placed = oracle.tap_place(lay["f"], lay["q_home"], lay["v_qo"], lay["kv_off"], lay["kv_grp"], lay["v_g"],
                              lay["resident"], lay["n_workers"])["sigma"]
    nt, W = len(placed), lay["n_workers"]
    scattered = np.array([(5 * t + 3) % W for t in range(nt)], np.int32)          # nearly every tile away from home
    return {"algorithm2": placed, "scattered": scattered, "home": lay["q_home"].astype(np.int32)}


@pytest.mark.parametrize("which,n_chunks", [("algorithm2", 4), ("scattered", 2), ("scattered", 4), ("home", 1)])
def test_executing_the_schedule_reproduces_the_single_pool_result(which, n_chunks):
    sigma = _sigmas()[which]
    world = (len(SEQ_OFF) - 1) * CP
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), sigma, n_chunks, out), nprocs=world, join=True)
    assert set(out.keys()) == set(range(world))
    f = {n: x.numpy() for n, x in _tensors().items()}
    o, lse = oracle.attn_fwd(f["q"], f["k"], f["v"], CU)
    dq, dk, dv = oracle.attn_bwd(f["q"], f["k"], f["v"], o, lse, f["dout"], CU)
    for r in range(world):
        res = out[r]
        t0, t1 = res["rows"]
        # rows are computed by the same per-row arithmetic wherever the tile runs: bit-identical
        assert np.array_equal(res["o"], o[t0:t1]) and np.array_equal(res["lse"], lse[:, t0:t1])
        assert np.array_equal(res["dq"], dq[t0:t1])
        # key gradients are sums of per-tile partial sums: equal up to the order of the additions
        for got, want in ((res["dk"], dk[t0:t1]), (res["dv"], dv[t0:t1])):
            assert np.abs(got - want).max() <= 2e-5 * max(1.0, np.abs(want).max())
