"""Error paths that must be reported, never executed: a malformed cu_seqlens, a planner that gives up, a plan used
on the wrong arguments.  Nothing here provokes a fault or a hang: the guards under test skip the work."""
import numpy as np
import pytest
import torch

from paper_2607_23250_b200 import pools

pytestmark = pytest.mark.gpu


def test_malformed_cu_seqlens_is_flagged_and_attention_does_no_work():
    from paper_2607_23250_b200 import binding as lb
    T, hq, hkv, d = 472, 2, 1, 128
    cu = torch.tensor([0, 5000, 100, T], dtype=torch.int32).cuda()        # not monotone, offset beyond T
    plan = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv, total_tokens=T)
    assert plan.status() == lb.ERR_BAD_SEQLENS
    t = pools.make_tensors(T, hq, hkv, d, seed=1, device="cuda")
    sentinel = 7.0
    out = torch.full_like(t["q"], sentinel)
    lse = torch.full((hq, T), sentinel, dtype=torch.float32, device="cuda")
    lb.libra_attn_pool_fwd(t["q"], t["k"], t["v"], plan, out=out, lse=lse)
    with pytest.raises(lb.LibraError) as err:
        plan.busy_times(lb.KERNEL_FWD)
    assert err.value.code == lb.ERR_BAD_SEQLENS
    assert bool((out == sentinel).all()) and bool((lse == sentinel).all())     # untouched
    dq, dk, dv = (torch.full_like(x, sentinel) for x in (t["q"], t["k"], t["v"]))
    lb.libra_attn_pool_bwd(t["q"], t["k"], t["v"], out, lse, t["dout"], plan, dq=dq, dk=dk, dv=dv)
    for kern in (lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        with pytest.raises(lb.LibraError) as err:
            plan.busy_times(kern)
        assert err.value.code == lb.ERR_BAD_SEQLENS
    for g in (dq, dk, dv):
        assert bool((g == sentinel).all())
    plan.destroy()
    # a good plan on the same GPU right afterwards works and reports OK
    cu = torch.tensor([0, 300, T], dtype=torch.int32).cuda()
    plan = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv)
    assert plan.status() == 0
    out, lse = lb.libra_attn_pool_fwd(t["q"], t["k"], t["v"], plan)
    plan.busy_times(lb.KERNEL_FWD)
    assert bool(torch.isfinite(out).all())
    plan.destroy()


def test_token_bounds_of_a_malformed_plan_stay_inside_the_pool():
    """The per-token sample bounds are clamped, so even the exported weights of a bad plan are finite sums."""
    from paper_2607_23250_b200 import binding as lb
    T = 1000
    cu = torch.tensor([0, 900000, 50, T], dtype=torch.int32).cuda()
    plan = lb.libra_plan_tiles(cu, 1, 256, tile_kv=128, n_heads_kv=1, total_tokens=T)
    assert plan.status() == lb.ERR_BAD_SEQLENS
    for direction in (lb.LIBRA_DIR_Q, lb.LIBRA_DIR_KV):
        w = plan.export(direction)["weight"]
        assert (w >= 0).all() and int(w.sum()) <= T * (T + 1) // 2
    plan.destroy()


def test_pool_planner_overflow_leaves_defined_outputs():
    """One sample so long that the integer soft-cap test could overflow: the planner reports OVERFLOW, every tile
    stays at its Q-home and the byte matrices stay zero.  Needs offsets only, no tensors."""
    from paper_2607_23250_b200 import binding as lb
    L = 1_200_000          # 64 shards x L (L + 1) / 2 pairs = 4.6e13 > the bound of about 4.4e13 at 1024 workers
    cu = torch.tensor([0, L], dtype=torch.int32).cuda()
    res = lb.libra_tap_plan(cu, [0, L], cp=1024, block=32768, n_shards=64, hq=64, hkv=4, head_dim=128)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == lb.ERR_OVERFLOW
    assert int(res["fwd_bytes"].abs().sum().item()) == 0 and int(res["bwd_bytes"].abs().sum().item()) == 0
    sigma = res["sigma"].cpu().numpy()
    assert sigma.min() >= 0 and sigma.max() < 1024


def test_plan_of_another_device_or_shape_is_refused():
    from paper_2607_23250_b200 import binding as lb
    cu = torch.tensor([0, 256], dtype=torch.int32).cuda()
    plan = lb.libra_plan_tiles(cu, 2, 256, tile_kv=128, n_heads_kv=1)
    q = torch.zeros((512, 2, 128), dtype=torch.bfloat16, device="cuda")         # T differs from the plan's
    k = torch.zeros((512, 1, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lb.LibraError) as err:
        lb.libra_attn_pool_fwd(q, k, k, plan)
    assert err.value.code == lb.ERR_PLAN_MISMATCH
    plan.destroy()


def test_bounded_wait_gives_up_and_reports_timeout():
    """The wait routine of the kernels, alone: a barrier nothing arrives on, nothing in flight.  It must give
    up after its budget, report TIMEOUT, and leave the GPU usable."""
    from paper_2607_23250_b200 import binding as lb
    for limit in (1_000, 2_000_000, 20_000_000):                  # 1 us, 2 ms, 20 ms
        st, waited = lb.libra_selftest_wait_timeout(limit)
        assert st == lb.ERR_TIMEOUT
        assert waited >= limit and waited < limit + 50_000_000    # not before the budget, not long after it
    x = torch.arange(8, device="cuda").sum().item()                # the context still works
    assert x == 28


def test_attention_kernels_give_up_cleanly_when_their_producer_stalls():
    """The failure is made on a healthy GPU by a flag that nothing sets: with the plan's stall injection on, the
    producer role issues no loads, so every consumer's wait runs out of its (shortened) budget.  Every CTA stops,
    frees its tensor memory and returns; the launch reports TIMEOUT.  With the injection off and the default
    budget restored the same plan gives correct results."""
    import oracle
    from paper_2607_23250_b200 import binding as lb
    lengths = [300, 200, 524]
    hq, hkv, d = 4, 2, 128
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, d, seed=3)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv)
    assert plan.status() == 0
    good_out, good_lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    plan.busy_times(lb.KERNEL_FWD)
    plan.set_wait_limit_ns(200_000)                                # 0.2 ms
    plan.inject_stall(True)
    lb.libra_attn_pool_fwd(q, k, v, plan)
    with pytest.raises(lb.LibraError) as err:
        plan.busy_times(lb.KERNEL_FWD)
    assert err.value.code == lb.ERR_TIMEOUT
    lb.libra_attn_pool_bwd(q, k, v, good_out, good_lse, dout, plan)
    with pytest.raises(lb.LibraError) as err:
        plan.busy_times(lb.KERNEL_BWD_DKDV)
    assert err.value.code == lb.ERR_TIMEOUT
    with pytest.raises(lb.LibraError) as err:
        plan.busy_times(lb.KERNEL_BWD_DQ)
    assert err.value.code == lb.ERR_TIMEOUT
    plan.inject_stall(False)
    plan.set_wait_limit_ns(0)                                      # back to the default budget
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    for kern in (lb.KERNEL_FWD, lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        plan.busy_times(kern)                                      # status words report the most recent launches: OK
    assert torch.equal(out, good_out) and torch.equal(lse, good_lse)
    f = {n: t[n].float().numpy() for n in t}
    o_ref, l_ref = oracle.attn_fwd(f["q"], f["k"], f["v"], cu_np)
    ref = oracle.attn_bwd(f["q"], f["k"], f["v"], o_ref, l_ref, f["dout"], cu_np)
    for g, r in zip((dq, dk, dv), ref):
        assert np.abs(g.float().cpu().numpy() - r).max() <= 5e-2 * np.abs(r).max()
    plan.destroy()


def test_fused_backward_gives_up_cleanly_when_its_producer_stalls():
    """The same injected stall for the fused backward (plan with pair tiles): TIMEOUT is reported, the context
    stays usable, and the next launch with the injection off is correct."""
    import oracle
    from paper_2607_23250_b200 import binding as lb
    lengths = [300, 200, 524]
    hq, hkv, d = 4, 2, 128
    cu_np = pools.cu_seqlens(lengths)
    t = pools.make_tensors(int(cu_np[-1]), hq, hkv, d, seed=4)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    plan = lb.libra_plan_tiles(torch.from_numpy(cu_np).cuda(), hq, 256, directions=lb.LIBRA_DIR_Q | lb.LIBRA_DIR_PAIR,
                               tile_kv=128, n_heads_kv=hkv)
    assert plan.status() == 0
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    plan.set_wait_limit_ns(200_000)                                # 0.2 ms
    plan.inject_stall(True)
    lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    with pytest.raises(lb.LibraError) as err:
        plan.busy_times(lb.KERNEL_BWD_FUSED)
    assert err.value.code == lb.ERR_TIMEOUT
    plan.inject_stall(False)
    plan.set_wait_limit_ns(0)
    dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    plan.busy_times(lb.KERNEL_BWD_FUSED)
    f = {n: t[n].float().numpy() for n in t}
    o_ref, l_ref = oracle.attn_fwd(f["q"], f["k"], f["v"], cu_np)
    ref = oracle.attn_bwd(f["q"], f["k"], f["v"], o_ref, l_ref, f["dout"], cu_np)
    for g, r in zip((dq, dk, dv), ref):
        assert np.abs(g.float().cpu().numpy() - r).max() <= 5e-2 * np.abs(r).max()
    plan.destroy()


def test_tile_times_cover_every_tile_that_ran():
    """Per-tile times of the forward (query-major tiles) and of the fused backward (pair tiles): every tile of the
    plan has run, so every entry is positive, and no tile took longer than the CTA that ran it was busy."""
    from paper_2607_23250_b200 import binding as lb
    lengths = [700, 1, 300, 129, 411, 2000]
    hq, hkv, d = 4, 2, 128
    cu_np = pools.cu_seqlens(lengths)
    t = pools.make_tensors(int(cu_np[-1]), hq, hkv, d, seed=5)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    plan = lb.libra_plan_tiles(torch.from_numpy(cu_np).cuda(), hq, 256, directions=lb.LIBRA_DIR_Q | lb.LIBRA_DIR_PAIR,
                               tile_kv=128, n_heads_kv=hkv)
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    for kern, direction in ((lb.KERNEL_FWD, lb.LIBRA_DIR_Q), (lb.KERNEL_BWD_FUSED, lb.LIBRA_DIR_PAIR)):
        ns = plan.tile_times(kern)
        busy = plan.busy_times(kern)
        ex = plan.export(direction)
        assert len(ns) == plan.info(direction)["n_tiles"] and (ns > 0).all()
        assert (ns.astype(np.int64) <= busy[ex["cta_of_tile"]].astype(np.int64)).all()
    with pytest.raises(lb.LibraError) as err:
        plan.tile_times(lb.KERNEL_BWD_DQ)
    assert err.value.code == lb.ERR_INVALID_ARG
    plan.destroy()
