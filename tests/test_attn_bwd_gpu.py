"""Backward pool attention (CUDA, through the C ABI) against the CPU oracle's gradient."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools
from parity import band_errors, rel_to_max

pytestmark = pytest.mark.gpu

TOL_G = 5e-2   # max-abs error relative to max magnitude (the benchmark's stated bound for dQ/dK/dV)


def _run(lengths, hq, hkv, d, seed=0, W=0, qscale=1.0, H=0):
    from paper_2607_23250_b200 import binding as lb
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, d, seed=seed, scale=qscale)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, H or hq, 256, n_workers=W, tile_kv=128, n_heads_kv=hkv)
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    plan.busy_times(lb.KERNEL_BWD_DKDV)                       # raises on a kernel timeout status
    plan.busy_times(lb.KERNEL_BWD_DQ)
    f = {n: t[n].float().numpy() for n in t}
    o_ref, l_ref = oracle.attn_fwd(f["q"], f["k"], f["v"], cu_np)
    ref = oracle.attn_bwd(f["q"], f["k"], f["v"], o_ref, l_ref, f["dout"], cu_np)
    got = [x.float().cpu().numpy() for x in (dq, dk, dv)]
    plan.destroy()
    return got, ref, cu_np


def _check(got, ref, cu):
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert np.isfinite(g).all(), name
        assert rel_to_max(g, r) <= TOL_G, (name, rel_to_max(g, r))
        assert band_errors(g, r, cu) <= TOL_G, (name, "band", band_errors(g, r, cu))


def test_tiny_config_full_parity():
    spec = pools.config(1)
    got, ref, cu = _run(pools.pool_lengths(spec), spec.hq, spec.hkv, spec.head_dim)
    _check(got, ref, cu)


@pytest.mark.parametrize("d", [64, 128])
def test_single_sample_multi_tile(d):
    got, ref, cu = _run([1000], 2, 1, d, seed=1)
    _check(got, ref, cu)


@pytest.mark.parametrize("seed", range(6))
def test_random_small_pools(seed):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(100, 2500))
    lengths = pools.random_layout(rng, T, int(rng.choice([3, 60, 300, 1200])))
    hkv = int(rng.choice([1, 2]))
    hq = hkv * int(rng.choice([1, 2, 4]))
    d = int(rng.choice([64, 128]))
    got, ref, cu = _run(lengths, hq, hkv, d, seed=seed, W=int(rng.choice([0, 3, 37])))
    _check(got, ref, cu)


@pytest.mark.parametrize("H,d,T", [(2, 128, 256 * 3 + 100), (1, 64, 256 * 2 + 129), (4, 128, 700), (1, 128, 128)])
def test_head_shards_wider_than_one_head(H, d, T):
    """Query-major tiles that carry several heads (units of one tile follow each other head by head), with a last
    tile whose second 128-row half is partly or wholly past the end of the pool."""
    rng = np.random.default_rng(T + H)
    lengths = pools.random_layout(rng, T, 400)
    got, ref, cu = _run(lengths, 4, 2, d, seed=11, H=H, W=int(rng.choice([0, 2, 5])))
    _check(got, ref, cu)


def test_boundary_lengths_and_three_samples_in_one_tile():
    lengths = [1, 127, 128, 129, 255, 257, 1, 1, 40, 50, 60, 300, 5]
    got, ref, cu = _run(lengths, 4, 2, 128, seed=3)
    _check(got, ref, cu)


def test_peaked_softmax():
    got, ref, cu = _run([700, 900], 2, 2, 64, seed=4, qscale=4.0)
    _check(got, ref, cu)


def test_single_token_pool():
    got, ref, cu = _run([1], 2, 1, 64, seed=6)
    # a length-1 sample has dQ = dK = 0 and dV = sum over the group of dO
    assert np.abs(got[0]).max() < 1e-6 and np.abs(got[1]).max() < 1e-6
    assert rel_to_max(got[2], ref[2]) <= TOL_G


@pytest.mark.parametrize("hq,hkv", [(64, 4), (128, 4)], ids=["G16", "G32"])
def test_wide_query_head_groups(hq, hkv):
    """Sixteen and thirty-two query heads per kv head at head_dim 128: dK / dV sum over the whole group."""
    got, ref, cu = _run([700, 1, 300, 129, 411], hq, hkv, 128, seed=31)
    _check(got, ref, cu)
