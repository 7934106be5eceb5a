"""The allocation-free backward entry point gives the same gradients as the regular one.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  Calls go through the C ABI; two calls in a row share the library's built-in
scratch and must both match.
"""
import numpy as np
import pytest
import torch

from paper_2607_23250_b200 import pools

pytestmark = pytest.mark.gpu


def _setup(lengths, hq, hkv, d, seed):
    from paper_2607_23250_b200 import binding as lb
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, d, seed=seed)
    q, k, v, dout = (t[n].cuda() for n in ("q", "k", "v", "dout"))
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv)
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    return lb, plan, (q, k, v, out, lse, dout)


def test_noalloc_backward_matches_regular_backward_twice():
    lb, plan, (q, k, v, out, lse, dout) = _setup([300, 1, 700, 129, 523, 90], 4, 2, 128, seed=21)
    ref = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)            # caller-provided workspace
    torch.cuda.synchronize()
    for call in range(2):                                                   # second call reuses the dirty scratch
        got = (torch.full_like(q, float("nan")), torch.full_like(k, float("nan")), torch.full_like(v, float("nan")))
        before = torch.cuda.memory_allocated()
        lb.libra_attn_pool_bwd_noalloc(q, k, v, out, lse, dout, plan, *got)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before                     # torch's allocator was not touched
        for name, g, r in zip(("dq", "dk", "dv"), got, ref):
            # same kernels, same order of additions, no atomics: the two entry points agree bit for bit
            assert torch.equal(g, r), (name, call)
    for kern in (lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ):
        plan.busy_times(kern)                                               # raises on a device-side timeout
    plan.destroy()


def test_noalloc_different_shape_after_first_use():
    # a second problem with another head_dim and a ragged tail, after the scratch holds other data
    lb, plan, (q, k, v, out, lse, dout) = _setup([65, 400, 7], 2, 1, 64, seed=22)
    ref = lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan)
    got = (torch.empty_like(q), torch.empty_like(k), torch.empty_like(v))
    lb.libra_attn_pool_bwd_noalloc(q, k, v, out, lse, dout, plan, *got)
    torch.cuda.synchronize()
    for name, g, r in zip(("dq", "dk", "dv"), got, ref):
        assert torch.equal(g, r), name
    plan.destroy()


def test_noalloc_reports_bad_dimensions_like_the_regular_call():
    from paper_2607_23250_b200 import binding as lb
    cu = torch.tensor([0, 256], dtype=torch.int32).cuda()
    plan = lb.libra_plan_tiles(cu, 2, 256, tile_kv=128, n_heads_kv=1)
    q = torch.zeros((256, 2, 96), dtype=torch.bfloat16, device="cuda")       # head_dim 96: no such kernel
    k = torch.zeros((256, 1, 96), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((2, 256), dtype=torch.float32, device="cuda")
    codes = []
    for call in (lambda: lb.libra_attn_pool_bwd(q, k, k, q, lse, q, plan, workspace=torch.empty(4096, dtype=torch.uint8, device="cuda")),
                 lambda: lb.libra_attn_pool_bwd_noalloc(q, k, k, q, lse, q, plan, torch.empty_like(q), torch.empty_like(k),
                                                        torch.empty_like(k))):
        with pytest.raises(lb.LibraError) as err:
            call()
        codes.append(err.value.code)
    assert codes == [lb.ERR_UNSUPPORTED, lb.ERR_UNSUPPORTED]
    plan.destroy()


def test_noalloc_rejects_pools_beyond_the_builtin_scratch():
    from paper_2607_23250_b200 import binding as lb
    limit = lb.libra_attn_pool_bwd_noalloc_max_bytes()
    assert limit == 16 * 1024 * 1024
    # 2 * hq * round_up(T, 128) * 4 bytes must exceed the limit: hq = 64, T = 40000 -> 20.5 MB
    T, hq, hkv, d = 40000, 64, 1, 64
    cu = torch.tensor([0, T], dtype=torch.int32).cuda()
    plan = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv)
    q = torch.zeros((T, hq, d), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((T, hkv, d), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((hq, T), dtype=torch.float32, device="cuda")
    assert lb.libra_attn_pool_bwd_workspace_bytes(plan, q, k) > limit
    n0 = lb.launch_count()
    with pytest.raises(lb.LibraError) as err:
        lb.libra_attn_pool_bwd_noalloc(q, k, k, q, lse, q, plan, torch.empty_like(q), torch.empty_like(k),
                                       torch.empty_like(k))
    assert err.value.code == lb.ERR_SCRATCH_TOO_SMALL
    assert lb.launch_count() == n0                                          # nothing was launched
    plan.destroy()
