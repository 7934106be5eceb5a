"""The exchange executor with the library's kernels: four CPU ranks (gloo) move the rows the schedule lists, chunk by
chunk, and every rank computes the tiles placed on it with the CUDA kernels (all four processes use GPU 0; their
kernels never wait on one another, only the host-side messages do).  The workers' outputs and gradients put together
agree with the oracle on the whole pool."""
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

pytestmark = pytest.mark.gpu

CU = [0, 200, 201, 700, 1024]
SEQ_OFF = [0, 512, 1024]             # P = 2 packed sequences x 512 tokens, CP = 2: runs of 256 tokens
CP, BLOCK, H, HQ, HKV, D = 2, 128, 2, 8, 2, 64


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _tensors():
    return pools.make_tensors(CU[-1], HQ, HKV, D, seed=21)          # bf16, the same on every rank


def _worker(rank, world, port, sigma, n_chunks, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    lay = exchange.PoolLayout(tuple(CU), tuple(SEQ_OFF), CP, BLOCK, H, HQ, HKV, D)
    rec = osched.schedule(CU, SEQ_OFF, CP, BLOCK, H, sigma)
    t0, t1 = lay.run(rank)
    local = {n: x[t0:t1].contiguous() for n, x in _tensors().items()}
    fwd, bwd = exchange.library_attention("cuda")
    w = exchange.Worker(rank, lay, sigma, rec, n_chunks, local, fwd, bwd, dist, torch)
    o, lse = w.forward()
    dq, dk, dv = w.backward()
    out[rank] = dict(rows=(t0, t1), o=o.float().numpy(), lse=lse.numpy(), dq=dq.float().numpy(), dk=dk.float().numpy(),
                     dv=dv.float().numpy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("which,n_chunks", [("algorithm2", 2), ("scattered", 4)])
def test_exchange_with_the_cuda_kernels_reproduces_the_pool(which, n_chunks):
    lay = oracle.tap_layout(CU, SEQ_OFF, CP, BLOCK, H, HQ, HKV, D)
    if which == "algorithm2":
        sigma = oracle.tap_place(lay["f"], lay["q_home"], lay["v_qo"], lay["kv_off"], lay["kv_grp"], lay["v_g"],
                                 lay["resident"], lay["n_workers"])["sigma"]
    else:
        sigma = np.array([(5 * t + 3) % lay["n_workers"] for t in range(len(lay["f"]))], np.int32)
    world = (len(SEQ_OFF) - 1) * CP
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(world, _free_port(), sigma, n_chunks, out), nprocs=world, join=True)
    assert set(out.keys()) == set(range(world))
    f = {n: x.float().numpy() for n, x in _tensors().items()}
    o, lse = oracle.attn_fwd(f["q"], f["k"], f["v"], CU)
    dq, dk, dv = oracle.attn_bwd(f["q"], f["k"], f["v"], o, lse, f["dout"], CU)
    for r in range(world):
        res = out[r]
        t0, t1 = res["rows"]
        assert np.abs(res["o"] - o[t0:t1]).max() <= 2e-2 * np.abs(o).max()
        assert np.abs(res["lse"] - lse[:, t0:t1]).max() <= 1e-3
        for got, want, full in ((res["dq"], dq[t0:t1], dq), (res["dk"], dk[t0:t1], dk), (res["dv"], dv[t0:t1], dv)):
            assert np.abs(got - want).max() <= 5e-2 * np.abs(full).max()
