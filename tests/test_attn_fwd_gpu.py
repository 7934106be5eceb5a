"""Forward pool attention (CUDA, through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools
from parity import band_errors, rel_to_max

pytestmark = pytest.mark.gpu

TOL_O = 2e-2      # max-abs error relative to max magnitude (the benchmark's stated bound)
TOL_LSE = 1e-3    # absolute; a dropped key block moves LSE by >= 1e-2


def _run(lengths, hq, hkv, d, seed=0, H=None, W=0, qscale=1.0, kshift=0.0):
    from paper_2607_23250_b200 import binding as lb
    cu_np = pools.cu_seqlens(lengths)
    T = int(cu_np[-1])
    t = pools.make_tensors(T, hq, hkv, d, seed=seed, scale=qscale)
    if kshift:
        t["k"] = (t["k"].float() + kshift).to(torch.bfloat16)
    q, k, v = (t[n].cuda() for n in ("q", "k", "v"))
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, H or hq, 256, n_workers=W, directions=lb.LIBRA_DIR_Q)
    out, lse = lb.libra_attn_pool_fwd(q, k, v, plan)
    torch.cuda.synchronize()
    st = lb._lib.libra_busy_times(plan._h, lb.KERNEL_FWD, np.zeros(plan.info()["n_workers"], np.uint64).ctypes.data_as(lb._vp))
    assert st == 0, f"kernel status {st}"
    o_ref, l_ref = oracle.attn_fwd(t["q"].float().numpy(), t["k"].float().numpy(), t["v"].float().numpy(), cu_np)
    o = out.float().cpu().numpy()
    l = lse.cpu().numpy()
    plan.destroy()
    return o, l, o_ref, l_ref, cu_np


def _check(o, l, o_ref, l_ref, cu):
    assert np.isfinite(o).all() and np.isfinite(l).all()
    assert rel_to_max(o, o_ref) <= TOL_O
    assert np.abs(l - l_ref).max() <= TOL_LSE
    assert band_errors(o, o_ref, cu) <= TOL_O


def test_tiny_config_full_parity():
    spec = pools.config(1)
    o, l, o_ref, l_ref, cu = _run(pools.pool_lengths(spec), spec.hq, spec.hkv, spec.head_dim)
    _check(o, l, o_ref, l_ref, cu)


@pytest.mark.parametrize("d", [64, 128])
def test_single_sample_multi_tile(d):
    o, l, o_ref, l_ref, cu = _run([1000], 2, 1, d, seed=1)
    _check(o, l, o_ref, l_ref, cu)


@pytest.mark.parametrize("seed", range(6))
def test_random_small_pools(seed):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(100, 2500))                       # ragged tails, several tiles
    lengths = pools.random_layout(rng, T, int(rng.choice([3, 60, 300, 1200])))
    hkv = int(rng.choice([1, 2]))
    hq = hkv * int(rng.choice([1, 2, 4]))
    d = int(rng.choice([64, 128]))
    H = int(rng.choice([h for h in (1, 2, 4, 8) if hq % h == 0]))
    o, l, o_ref, l_ref, cu = _run(lengths, hq, hkv, d, seed=seed, H=H, W=int(rng.choice([0, 3, 37])))
    _check(o, l, o_ref, l_ref, cu)


def test_boundary_lengths_and_three_samples_in_one_tile():
    lengths = [1, 127, 128, 129, 255, 257, 1, 1, 40, 50, 60, 300, 5]
    o, l, o_ref, l_ref, cu = _run(lengths, 4, 2, 128, seed=3)
    _check(o, l, o_ref, l_ref, cu)


def test_peaked_softmax_and_score_offset():
    # Q scaled x8 makes the running max move a lot (exercises the O rescale path)
    o, l, o_ref, l_ref, cu = _run([700, 900], 2, 2, 64, seed=4, qscale=8.0)
    _check(o, l, o_ref, l_ref, cu)
    # a constant added to every key shifts scores by q.c: large, row-dependent offsets
    o, l, o_ref, l_ref, cu = _run([512, 300], 2, 1, 128, seed=5, kshift=3.0)
    assert rel_to_max(o, o_ref) <= TOL_O
    assert np.abs(l - l_ref).max() <= 2e-2 * max(1.0, np.abs(l_ref).max() / 50)


def test_single_token_pool():
    o, l, o_ref, l_ref, cu = _run([1], 1, 1, 64, seed=6)
    _check(o, l, o_ref, l_ref, cu)


@pytest.mark.parametrize("hq,hkv", [(64, 4), (128, 4)], ids=["G16", "G32"])
def test_wide_query_head_groups(hq, hkv):
    """Sixteen and thirty-two query heads per kv head (the 235B-shaped and the micro-benchmark head counts of
    the paper's Table 1) at head_dim 128, several samples, ragged tail."""
    o, l, o_ref, l_ref, cu = _run([700, 1, 300, 129, 411], hq, hkv, 128, seed=31, H=hq // 2)
    _check(o, l, o_ref, l_ref, cu)
