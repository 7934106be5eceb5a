"""head_dim 256 (the micro-benchmark head shape, Table 1): forward and backward against the CPU oracle.  `pairs` runs
the dV and dK passes over the plan's pair tiles (fp32 accumulators) instead of its key-major tiles."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools
from parity import band_errors, rel_to_max

pytestmark = pytest.mark.gpu

TOL_O, TOL_G, TOL_LSE = 2e-2, 5e-2, 1e-3
D = 256


def _run(lengths, hq, hkv, seed=0, W=0, H=0, qscale=1.0, backward=True, pairs=False, chunk=0):
    from paper_2607_23250_b200 import binding as lb
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, D, seed=seed, scale=qscale)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    cu = torch.from_numpy(cu_np).cuda()
    directions = lb.LIBRA_DIR_Q | (lb.LIBRA_DIR_PAIR if pairs else lb.LIBRA_DIR_KV)
    plan = lb.libra_plan_tiles(cu, H or hq, 256, n_workers=W, directions=directions, tile_kv=128, n_heads_kv=hkv,
                               pair_chunk=chunk)
    assert plan.status() == 0
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    torch.cuda.synchronize()
    plan.busy_times(lb.KERNEL_FWD)                            # raises on a kernel timeout status
    got = dict(out=out.float().cpu().numpy(), lse=lse.cpu().numpy())
    f = {n: t[n].float().numpy() for n in t}
    o_ref, l_ref = oracle.attn_fwd(f["q"], f["k"], f["v"], cu_np)
    ref = dict(out=o_ref, lse=l_ref)
    if backward:
        dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
        torch.cuda.synchronize()
        plan.busy_times(lb.KERNEL_BWD_FUSED if pairs else lb.KERNEL_BWD_DKDV)
        plan.busy_times(lb.KERNEL_BWD_DQ)
        got.update(dq=dq.float().cpu().numpy(), dk=dk.float().cpu().numpy(), dv=dv.float().cpu().numpy())
        ref.update(zip(("dq", "dk", "dv"), oracle.attn_bwd(f["q"], f["k"], f["v"], o_ref, l_ref, f["dout"], cu_np)))
    plan.destroy()
    return got, ref, cu_np


def _check(got, ref, cu):
    assert rel_to_max(got["out"], ref["out"]) <= TOL_O, rel_to_max(got["out"], ref["out"])
    assert np.abs(got["lse"] - ref["lse"]).max() <= TOL_LSE
    assert band_errors(got["out"], ref["out"], cu) <= TOL_O
    for name in ("dq", "dk", "dv"):
        if name in got:
            assert np.isfinite(got[name]).all(), name
            assert rel_to_max(got[name], ref[name]) <= TOL_G, (name, rel_to_max(got[name], ref[name]))
            assert band_errors(got[name], ref[name], cu) <= TOL_G, (name, "band")


def test_one_block():
    _check(*_run([64], 1, 1, seed=1))


@pytest.mark.parametrize("pairs", [False, True])
def test_single_sample_multi_tile(pairs):
    _check(*_run([1000], 2, 1, seed=2, pairs=pairs, chunk=256))


@pytest.mark.parametrize("pairs", [False, True])
def test_tiny_layout(pairs):
    spec = pools.config(1)      # the 4096-token layout of the full-parity config, at this head width
    _check(*_run(pools.pool_lengths(spec), 4, 2, seed=3, pairs=pairs))


@pytest.mark.parametrize("pairs", [False, True])
@pytest.mark.parametrize("seed", range(5))
def test_random_small_pools(seed, pairs):
    rng = np.random.default_rng(200 + seed)
    T = int(rng.integers(100, 2500))
    lengths = pools.random_layout(rng, T, int(rng.choice([3, 60, 300, 1200])))
    hkv = int(rng.choice([1, 2]))
    hq = hkv * int(rng.choice([1, 2, 4]))
    _check(*_run(lengths, hq, hkv, seed=seed, W=int(rng.choice([0, 3, 37])), pairs=pairs,
                 chunk=int(rng.choice([0, 128, 512]))))


@pytest.mark.parametrize("pairs", [False, True])
def test_boundary_lengths_and_ragged_end(pairs):
    _check(*_run([1, 63, 64, 65, 127, 128, 129, 255, 257, 1, 1, 40, 50, 60, 300, 5], 4, 2, seed=4, pairs=pairs))


@pytest.mark.parametrize("pairs", [False, True])
def test_microbenchmark_head_shape(pairs):
    """Hq 128 / Hkv 4: thirty-two query heads per kv head."""
    _check(*_run([700, 1, 300, 129, 411], 128, 4, seed=5, pairs=pairs))


def test_head_shards_wider_than_one_head():
    _check(*_run([900, 256 * 2 + 100], 4, 2, seed=6, H=2, W=5))


def test_peaked_softmax():
    _check(*_run([700, 900], 2, 2, seed=7, qscale=3.0))


def test_single_token_pool():
    got, ref, cu = _run([1], 2, 1, seed=8)
    assert np.abs(got["dq"]).max() < 1e-6 and np.abs(got["dk"]).max() < 1e-6
    assert rel_to_max(got["dv"], ref["dv"]) <= TOL_G
    assert rel_to_max(got["out"], ref["out"]) <= TOL_O


@pytest.mark.parametrize("pairs", [False, True])
def test_sampled_rows_of_a_long_sample(pairs):
    """A 32768-token sample beside short ones: sampled rows of O / LSE / dQ and key columns of dK / dV recomputed by
    the oracle one by one (the whole sample would take it minutes)."""
    from paper_2607_23250_b200 import binding as lb
    lengths = [300, 32768, 1000]
    hq, hkv = 4, 2
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, D, seed=9, device="cuda")
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, hq, 256, directions=lb.LIBRA_DIR_Q | (lb.LIBRA_DIR_PAIR if pairs else lb.LIBRA_DIR_KV),
                               tile_kv=128, n_heads_kv=hkv)
    out, lse = lb.libra_attn_pool_fwd(t["q"], t["k"], t["v"], plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(t["q"], t["k"], t["v"], out, lse, t["dout"], plan)
    torch.cuda.synchronize()
    for kern in (lb.KERNEL_FWD, lb.KERNEL_BWD_FUSED if pairs else lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        plan.busy_times(kern)
    s, e, n = int(cu_np[1]), int(cu_np[2]), lengths[1]
    G = hq // hkv
    f = lambda x: x.float().cpu().numpy()
    rng = np.random.default_rng(0)
    rows = np.array(sorted({0, 1, 63, 64, 127, 128, 255, 256, n // 2, n - 129, n - 2, n - 1} | {int(x) for x in rng.integers(0, n, 4)}))
    zeros = np.zeros(len(rows), np.int32)
    kvh = 1
    dk_ref = np.zeros((len(rows), D)); dv_ref = np.zeros((len(rows), D))
    for g in range(G):
        h = kvh * G + g
        sub = dict(q=f(t["q"][s:e, h:h + 1]), k=f(t["k"][s:e, kvh:kvh + 1]), v=f(t["v"][s:e, kvh:kvh + 1]),
                   dout=f(t["dout"][s:e, h:h + 1]), out=f(out[s:e, h:h + 1]), lse=lse[h:h + 1, s:e].cpu().numpy())
        o_ref, l_ref = oracle.attn_fwd_rows(sub["q"], sub["k"], sub["v"], [0, n], rows, zeros)
        dq_ref = oracle.attn_dq_rows(sub["q"], sub["k"], sub["v"], sub["dout"], [0, n], rows, zeros)
        got_o, got_dq = f(out[s:e, h]), f(dq[s:e, h])
        for x, r in enumerate(rows):
            assert np.abs(got_o[r] - o_ref[x]).max() <= TOL_O * max(np.abs(o_ref[x]).max(), 1e-3)
            assert abs(float(sub["lse"][0, r]) - float(l_ref[x])) <= TOL_LSE
            assert np.abs(got_dq[r] - dq_ref[x]).max() <= TOL_G * max(np.abs(dq_ref[x]).max(), 1e-2)
        a, b = oracle.attn_dkv_cols(sub["q"], sub["k"], sub["v"], sub["out"], sub["lse"], sub["dout"], [0, n], rows, zeros)
        dk_ref += a
        dv_ref += b
    got_dk, got_dv = f(dk[s:e, kvh]), f(dv[s:e, kvh])
    for x, c in enumerate(rows):
        assert np.abs(got_dk[c] - dk_ref[x]).max() <= TOL_G * max(np.abs(dk_ref[x]).max(), 1e-2), ("dk", int(c))
        assert np.abs(got_dv[c] - dv_ref[x]).max() <= TOL_G * max(np.abs(dv_ref[x]).max(), 1e-2), ("dv", int(c))
    plan.destroy()


def test_give_up_path_of_the_256_wide_kernel():
    """Producer stall injected on a healthy GPU (no loads are issued, a flag nothing sets): every pass reports
    TIMEOUT through the status words and returns; with the injection off the same plan gives correct results."""
    from paper_2607_23250_b200 import binding as lb
    lengths = [300, 200, 524]
    hq, hkv = 4, 2
    cu_np = pools.cu_seqlens(lengths)
    t = pools.make_tensors(int(cu_np[-1]), hq, hkv, D, seed=12)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    plan = lb.libra_plan_tiles(torch.from_numpy(cu_np).cuda(), hq, 256, tile_kv=128, n_heads_kv=hkv)
    good_out, good_lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    plan.busy_times(lb.KERNEL_FWD)
    plan.set_wait_limit_ns(200_000)
    plan.inject_stall(True)
    lb.libra_attn_pool_fwd(q, k, v, plan)
    with pytest.raises(lb.LibraError) as err:
        plan.busy_times(lb.KERNEL_FWD)
    assert err.value.code == lb.ERR_TIMEOUT
    lb.libra_attn_pool_bwd(q, k, v, good_out, good_lse, dout, plan)
    for kern in (lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        with pytest.raises(lb.LibraError) as err:
            plan.busy_times(kern)
        assert err.value.code == lb.ERR_TIMEOUT
    plan.inject_stall(False)
    plan.set_wait_limit_ns(0)
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    for kern in (lb.KERNEL_FWD, lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        plan.busy_times(kern)
    assert torch.equal(out, good_out) and torch.equal(lse, good_lse)
    f = {n: t[n].float().numpy() for n in t}
    o_ref, l_ref = oracle.attn_fwd(f["q"], f["k"], f["v"], cu_np)
    ref = oracle.attn_bwd(f["q"], f["k"], f["v"], o_ref, l_ref, f["dout"], cu_np)
    for g, r in zip((dq, dk, dv), ref):
        assert np.abs(g.float().cpu().numpy() - r).max() <= TOL_G * np.abs(r).max()
    plan.destroy()
