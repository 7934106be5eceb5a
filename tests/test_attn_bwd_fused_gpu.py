"""Fused backward (one kernel over the plan's pair tiles, five GEMMs per cell, fp32 accumulators) against the CPU
oracle's gradient.  The call is the same libra_attn_pool_bwd; the plan carries pair tiles, which selects this form."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools
from parity import band_errors, rel_to_max

pytestmark = pytest.mark.gpu

TOL_G = 5e-2   # max-abs error relative to max magnitude (the benchmark's stated bound for dQ/dK/dV)


def _run(lengths, hq, hkv, d=128, seed=0, W=0, qscale=1.0, chunk=0, with_kv=False, repeat=False):
    from paper_2607_23250_b200 import binding as lb
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, d, seed=seed, scale=qscale)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    cu = torch.from_numpy(cu_np).cuda()
    directions = lb.LIBRA_DIR_Q | lb.LIBRA_DIR_PAIR | (lb.LIBRA_DIR_KV if with_kv else 0)
    plan = lb.libra_plan_tiles(cu, hq, 256, n_workers=W, directions=directions, tile_kv=128, n_heads_kv=hkv,
                               pair_chunk=chunk)
    assert plan.status() == 0
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    if d == 128:
        plan.busy_times(lb.KERNEL_BWD_FUSED)                  # raises on a kernel timeout status
        assert len(plan.kernel_times_ms(lb.KERNEL_BWD_FUSED)) == 0   # timing is off unless asked for
    again = None
    if repeat:
        again = [x.float().cpu().numpy() for x in lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)]
    f = {n: t[n].float().numpy() for n in t}
    o_ref, l_ref = oracle.attn_fwd(f["q"], f["k"], f["v"], cu_np)
    ref = oracle.attn_bwd(f["q"], f["k"], f["v"], o_ref, l_ref, f["dout"], cu_np)
    got = [x.float().cpu().numpy() for x in (dq, dk, dv)]
    plan.destroy()
    return got, ref, cu_np, again


def _check(got, ref, cu):
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert np.isfinite(g).all(), name
        assert rel_to_max(g, r) <= TOL_G, (name, rel_to_max(g, r))
        assert band_errors(g, r, cu) <= TOL_G, (name, "band", band_errors(g, r, cu))


def test_tiny_layout_full_parity():
    spec = pools.config(1)          # the 4096-token layout; the fused form exists for head_dim 128 only
    got, ref, cu, _ = _run(pools.pool_lengths(spec), spec.hq, spec.hkv, 128)
    _check(got, ref, cu)


@pytest.mark.parametrize("chunk", [128, 256, 512, 2048])
def test_query_chunk_sizes(chunk):
    """One sample over several key blocks and query chunks; chunk 128 makes every pair tile a single cell."""
    got, ref, cu, _ = _run([1000, 37, 900], 4, 2, seed=1, chunk=chunk)
    _check(got, ref, cu)


@pytest.mark.parametrize("seed", range(6))
def test_random_small_pools(seed):
    rng = np.random.default_rng(100 + seed)
    T = int(rng.integers(100, 2500))
    lengths = pools.random_layout(rng, T, int(rng.choice([3, 60, 300, 1200])))
    hkv = int(rng.choice([1, 2]))
    hq = hkv * int(rng.choice([1, 2, 4]))
    got, ref, cu, _ = _run(lengths, hq, hkv, seed=seed, W=int(rng.choice([0, 3, 37])),
                           chunk=int(rng.choice([0, 256, 1024])))
    _check(got, ref, cu)


def test_boundary_lengths_and_three_samples_in_one_block():
    lengths = [1, 127, 128, 129, 255, 257, 1, 1, 40, 50, 60, 300, 5]
    got, ref, cu, _ = _run(lengths, 4, 2, seed=3)
    _check(got, ref, cu)


def test_ragged_last_block():
    """The pool ends inside a key block: rows past the end contribute nothing and are never written."""
    got, ref, cu, _ = _run([256 * 3 + 100], 2, 1, seed=7, chunk=512)
    _check(got, ref, cu)


def test_peaked_softmax():
    got, ref, cu, _ = _run([700, 900], 2, 2, seed=4, qscale=4.0)
    _check(got, ref, cu)


def test_single_token_pool():
    got, ref, cu, _ = _run([1], 2, 1, seed=6)
    # a length-1 sample has dQ = dK = 0 and dV = sum over the group of dO
    assert np.abs(got[0]).max() < 1e-6 and np.abs(got[1]).max() < 1e-6
    assert rel_to_max(got[2], ref[2]) <= TOL_G


@pytest.mark.parametrize("hq,hkv", [(64, 4), (128, 4)], ids=["G16", "G32"])
def test_wide_query_head_groups(hq, hkv):
    got, ref, cu, _ = _run([700, 1, 300, 129, 411], hq, hkv, seed=31)
    _check(got, ref, cu)


def test_more_workers_than_tiles_and_one_worker():
    for W in (1, 148):
        got, ref, cu, _ = _run([300, 200], 2, 1, seed=8, W=W)
        _check(got, ref, cu)


def test_repeat_agrees_to_rounding_and_kv_lists_are_ignored():
    """The additions into the fp32 accumulators come in a different order on every run: two runs agree to the
    rounding of the final bf16 conversion, not bit for bit.  A plan that also carries key-major lists still takes
    the fused form."""
    got, ref, cu, again = _run([1500, 800, 64], 8, 2, seed=9, with_kv=True, repeat=True)
    _check(got, ref, cu)
    for g, a in zip(got, again):
        assert np.abs(g - a).max() <= 2.0 ** -7 * max(np.abs(g).max(), 1e-6)


def test_head_dim_64_falls_back_to_the_two_kernel_form():
    got, ref, cu, _ = _run([700, 300], 4, 2, d=64, seed=10, with_kv=True)
    _check(got, ref, cu)


def test_fused_needs_no_key_major_lists_but_head_dim_64_does():
    from paper_2607_23250_b200 import binding as lb
    cu_np = pools.cu_seqlens([300])
    t = pools.make_tensors(300, 2, 1, 64, seed=0)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    plan = lb.libra_plan_tiles(torch.from_numpy(cu_np).cuda(), 2, 256, directions=lb.LIBRA_DIR_Q | lb.LIBRA_DIR_PAIR,
                               tile_kv=128, n_heads_kv=1)
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    with pytest.raises(lb.LibraError) as e:
        lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    assert e.value.code == lb.ERR_PLAN_MISMATCH
    plan.destroy()
