"""Head-sharded execution on one GPU: the N head slices of a pool, run one after another through the C ABI,
put together equal the unsharded call bit for bit (heads are independent and every result is computed by
the same instruction sequence whichever CTA runs its tile)."""
import numpy as np
import pytest
import torch

from paper_2607_23250_b200 import pools, sharding

pytestmark = pytest.mark.gpu


def _run(lb, cu, q, k, v, dout):
    hq, hkv = q.shape[1], k.shape[1]
    plan = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv)
    assert plan.status() == 0
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    torch.cuda.synchronize()
    for kern in (lb.KERNEL_FWD, lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        plan.busy_times(kern)
    plan.destroy()
    return out, lse, dq, dk, dv


@pytest.mark.parametrize("hq,hkv,world", [(8, 4, 2), (8, 4, 4), (8, 2, 4)], ids=["2_ranks", "4_ranks", "kv_head_shared"])
def test_head_slices_reproduce_the_unsharded_call(hq, hkv, world):
    from paper_2607_23250_b200 import binding as lb
    lengths = [700, 1, 300, 129, 411, 260]
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, 128, seed=41, device="cuda")
    cu = torch.from_numpy(cu_np).cuda()
    out, lse, dq, dk, dv = _run(lb, cu, t["q"], t["k"], t["v"], t["dout"])
    dk_sum = torch.zeros_like(dk, dtype=torch.float32)
    dv_sum = torch.zeros_like(dv, dtype=torch.float32)
    shared = world > hkv
    for r in range(world):
        s = sharding.head_groups(hq, hkv, world, r)
        qs, ks, vs, dos = sharding.slice_heads(s, t["q"], t["k"], t["v"], t["dout"])
        o_r, l_r, dq_r, dk_r, dv_r = _run(lb, cu, qs, ks, vs, dos)
        qh, kh = list(s.q_heads), list(s.kv_heads)
        assert torch.equal(o_r, out[:, qh]) and torch.equal(l_r, lse[qh]) and torch.equal(dq_r, dq[:, qh])
        if not shared:
            assert torch.equal(dk_r, dk[:, kh]) and torch.equal(dv_r, dv[:, kh])
        else:
            dk_sum[:, kh] += dk_r.float()
            dv_sum[:, kh] += dv_r.float()
    if shared:     # partial sums over the query heads of a kv head, added as the sub-group all-reduce would
        for got, want in ((dk_sum, dk.float()), (dv_sum, dv.float())):
            assert float((got - want).abs().max()) <= 2e-2 * float(want.abs().max())


def test_head_slices_with_the_fused_backward():
    """The same with pair-tile plans, i.e. the fused backward the benchmark runs per rank: its fp32 accumulation order
    varies from run to run, so the slices agree with the unsharded call to rounding (forward still bit for bit)."""
    from paper_2607_23250_b200 import binding as lb
    lengths = [700, 1, 300, 129, 411, 260]
    hq, hkv, world = 8, 4, 4
    cu_np = pools.cu_seqlens(lengths)
    t = pools.make_tensors(int(cu_np[-1]), hq, hkv, 128, seed=43, device="cuda")
    cu = torch.from_numpy(cu_np).cuda()

    def run(q, k, v, dout):
        plan = lb.libra_plan_tiles(cu, q.shape[1], 256, directions=lb.LIBRA_DIR_Q | lb.LIBRA_DIR_PAIR, tile_kv=128,
                                   n_heads_kv=k.shape[1])
        out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
        dq, dk, dv = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
        torch.cuda.synchronize()
        plan.busy_times(lb.KERNEL_BWD_FUSED)
        plan.destroy()
        return out, lse, dq, dk, dv

    out, lse, dq, dk, dv = run(t["q"], t["k"], t["v"], t["dout"])
    for r in range(world):
        s = sharding.head_groups(hq, hkv, world, r)
        qs, ks, vs, dos = sharding.slice_heads(s, t["q"], t["k"], t["v"], t["dout"])
        o_r, l_r, dq_r, dk_r, dv_r = run(qs, ks, vs, dos)
        qh, kh = list(s.q_heads), list(s.kv_heads)
        assert torch.equal(o_r, out[:, qh]) and torch.equal(l_r, lse[qh])
        for got, want in ((dq_r, dq[:, qh]), (dk_r, dk[:, kh]), (dv_r, dv[:, kh])):
            assert float((got.float() - want.float()).abs().max()) <= 2.0 ** -7 * float(want.float().abs().max())
