"""Full-size parity: the Qwen3-8B-shaped pool in the launch configuration the benchmark times, the 30B-shaped
pool with Pareto-tailed samples, the 1M-token pool with one 262144-token sample (Hq 64 / Hkv 4: sixteen query
heads per kv head, tensors beyond 2^32 bytes) and the skew sweep of 65536-token sequences at every skew.  The
"fused" cases run the same pools with a pair-tile plan, which makes the backward call take its fused form; config 6 is
the micro-benchmark head shape (Hq 128 / Hkv 4 / d 256) on two packed 32768-token sequences.

The whole oracle would take minutes here, so outputs are sampled: rows of O / LSE / dQ and
columns of dK / dV are recomputed one by one by the CPU oracle on the (sample, kv-head group)
sub-problem they belong to.  Short samples are checked with the oracle's own forward results
(the mathematical gradient); key columns of long samples use the out / lse arrays that are the
backward's inputs.  Properties that hold at any size are checked over the whole tensors.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools

pytestmark = pytest.mark.gpu

TOL_O, TOL_G, TOL_LSE = 2e-2, 5e-2, 1e-3


def _rel(got, want, floor=1e-3):
    want = np.asarray(want, np.float64)
    return float(np.abs(np.asarray(got, np.float64) - want).max() / max(np.abs(want).max(), floor))


@pytest.fixture(scope="module",
                params=[(2, 0.0, False), (2, 0.0, True), (3, 0.0, False), (3, 0.0, True), (4, 0.0, False), (4, 0.0, True),
                        (5, 0.0, False), (5, 0.25, False), (5, 0.5, False), (5, 1.0, False), (5, 1.0, True),
                        (6, 0.0, False), (6, 0.0, True)],
                ids=["config2", "config2_fused", "config3", "config3_fused", "config4", "config4_fused",
                     "config5_skew0", "config5_skew0.25", "config5_skew0.5", "config5_skew1", "config5_skew1_fused",
                     "config6_d256", "config6_d256_pairs"])
def run(request):
    from paper_2607_23250_b200 import binding as lb
    fused = request.param[2]
    spec = pools.config(*request.param[:2])
    lengths = pools.pool_lengths(spec)
    cu_np = pools.cu_seqlens(lengths)
    T, hq, hkv, d = spec.total_tokens, spec.hq, spec.hkv, spec.head_dim
    t = pools.make_tensors(T, hq, hkv, d, seed=0, device="cuda")
    cu = torch.from_numpy(cu_np).cuda()
    directions = lb.LIBRA_DIR_Q | (lb.LIBRA_DIR_PAIR if fused else lb.LIBRA_DIR_KV)
    plan = lb.libra_plan_tiles(cu, hq, 256, directions=directions, tile_kv=128, n_heads_kv=hkv,
                               total_tokens=T)                                             # as bench.py
    assert plan.status() == 0
    out, lse = lb.libra_attn_pool_fwd(t["q"], t["k"], t["v"], plan)
    dq, dk, dv = lb.libra_attn_pool_bwd(t["q"], t["k"], t["v"], out, lse, t["dout"], plan)
    torch.cuda.synchronize()
    for kern in (lb.KERNEL_FWD,) + ((lb.KERNEL_BWD_FUSED,) if fused else (lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ)):
        plan.busy_times(kern)
    if fused and d == 256:
        plan.busy_times(lb.KERNEL_BWD_DQ)       # at this width the dQ pass still walks the query-major lists
    res = dict(fused=fused, spec=spec, lengths=lengths, cu=cu_np, t=t, out=out, lse=lse, dq=dq, dk=dk, dv=dv, plan=plan, lb=lb)
    yield res
    plan.destroy()
    del res
    torch.cuda.empty_cache()


def _sub(run, j, kvh, heads=None, lo=0):
    """Host copy (fp32) of rows [lo, n) of sample j restricted to kv head kvh and the listed query heads of its
    group (offsets inside the group; default: the whole group)."""
    spec, cu, t = run["spec"], run["cu"], run["t"]
    G = spec.hq // spec.hkv
    s, e = int(cu[j]) + lo, int(cu[j + 1])
    hs = [kvh * G + g for g in (range(G) if heads is None else heads)]
    f = lambda x: x.float().cpu().numpy()
    return dict(q=f(t["q"][s:e, hs]), dout=f(t["dout"][s:e, hs]), k=f(t["k"][s:e, kvh:kvh + 1]),
                v=f(t["v"][s:e, kvh:kvh + 1]), out=f(run["out"][s:e, hs]), lse=run["lse"][hs, s:e].cpu().numpy(),
                dq=f(run["dq"][s:e, hs]), dk=f(run["dk"][s:e, kvh:kvh + 1]), dv=f(run["dv"][s:e, kvh:kvh + 1]),
                n=e - s, G=len(hs))


def test_plan_matches_oracle_at_full_size(run):
    lb, plan, spec = run["lb"], run["plan"], run["spec"]
    for direction, d_or, tile, H in ((lb.LIBRA_DIR_Q, 0, 256, spec.hq), (lb.LIBRA_DIR_KV, 1, 128, spec.hkv)):
        if direction == lb.LIBRA_DIR_KV and run["fused"]:
            continue
        got = plan.export(direction)
        want = oracle.plan(run["cu"], H, tile, plan.info(direction)["n_workers"], d_or)
        for key in ("weight", "order", "cta_of_tile", "cta_offsets", "cta_tiles", "loads"):
            assert np.array_equal(got[key], want[key]), (direction, key)


def test_sampled_rows_forward_and_dq(run):
    rng = np.random.default_rng(0)
    lengths = np.asarray(run["lengths"])
    order = np.argsort(-lengths)
    picks = list(order[:3]) + list(rng.choice(len(lengths), 5, replace=False))     # long samples and random ones
    G = run["spec"].hq // run["spec"].hkv
    worst = dict(o=0.0, lse=0.0, dq=0.0)
    for j in picks:
        kvh = int(rng.integers(0, run["spec"].hkv))
        n = int(lengths[j])
        cand = {0, n - 1, min(n - 1, 127), min(n - 1, 128), min(n - 1, 255), min(n - 1, 256), n // 2}
        cand |= {int(x) for x in rng.integers(0, n, 4)}
        # global tile boundaries that fall inside the sample
        first = int(run["cu"][j])
        cand |= {b - first for b in range((first // 256 + 1) * 256 - 1, first + n, max(4096, n // 8 // 256 * 256)) if 0 <= b - first < n}
        cand |= {b + 1 for b in list(cand) if b + 1 < n and (first + b + 1) % 256 == 0}
        rows = np.array(sorted(cand), dtype=np.int64)
        # one query head at a time keeps the host copy of a 262144-token sample at 134 MB per tensor
        for g in sorted({0, G - 1, int(rng.integers(0, G))})[: (3 if n <= 40000 else 2)]:
            s = _sub(run, int(j), kvh, heads=[g])
            zeros = np.zeros(len(rows), np.int32)
            o_ref, l_ref = oracle.attn_fwd_rows(s["q"], s["k"], s["v"], [0, n], rows, zeros)
            dq_ref = oracle.attn_dq_rows(s["q"], s["k"], s["v"], s["dout"], [0, n], rows, zeros)
            for x, r in enumerate(rows):
                worst["o"] = max(worst["o"], _rel(s["out"][r, 0], o_ref[x]))
                worst["lse"] = max(worst["lse"], abs(float(s["lse"][0, r]) - float(l_ref[x])))
                worst["dq"] = max(worst["dq"], _rel(s["dq"][r, 0], dq_ref[x], floor=1e-2))
    assert worst["o"] <= TOL_O and worst["lse"] <= TOL_LSE and worst["dq"] <= TOL_G, worst


def test_short_samples_full_gradient(run):
    """Samples of at most 1500 tokens: the whole sample against the oracle's own forward + backward."""
    rng = np.random.default_rng(1)
    lengths = np.asarray(run["lengths"])
    small = [j for j in range(len(lengths)) if 2 <= lengths[j] <= 1500]
    if not small:
        pytest.skip("the pool has no short samples")
    for j in rng.choice(small, min(4, len(small)), replace=False):
        kvh = int(rng.integers(0, run["spec"].hkv))
        s = _sub(run, int(j), kvh)
        cu = [0, s["n"]]
        o_ref, l_ref = oracle.attn_fwd(s["q"], s["k"], s["v"], cu)
        g_ref = oracle.attn_bwd(s["q"], s["k"], s["v"], o_ref, l_ref, s["dout"], cu)
        assert _rel(s["out"], o_ref) <= TOL_O
        assert np.abs(s["lse"] - l_ref).max() <= TOL_LSE
        for name, ref in zip(("dq", "dk", "dv"), g_ref):
            assert _rel(s[name], ref) <= TOL_G, (name, int(j))


def test_sampled_key_columns_of_long_samples(run):
    rng = np.random.default_rng(2)
    lengths = np.asarray(run["lengths"])
    G = run["spec"].hq // run["spec"].hkv
    for j in np.argsort(-lengths)[:2]:
        kvh = int(rng.integers(0, run["spec"].hkv))
        n = int(lengths[j])
        cols = np.array(sorted({0, 1, 127, 128, n // 3, n // 2, n - 129, n - 2, n - 1} & set(range(n))
                               | {int(x) for x in rng.integers(0, n, 3)}), dtype=np.int64)
        # a key column sums over the group's query heads: add the per-head columns (one head on the host at a time)
        dk_ref = np.zeros((len(cols), run["spec"].head_dim), np.float64)
        dv_ref = np.zeros_like(dk_ref)
        got = None
        for g in range(G):
            s = _sub(run, int(j), kvh, heads=[g])
            a, b = oracle.attn_dkv_cols(s["q"], s["k"], s["v"], s["out"], s["lse"], s["dout"], [0, n], cols,
                                        np.zeros(len(cols), np.int32))
            dk_ref += a
            dv_ref += b
            got = s
        for x, cidx in enumerate(cols):
            assert _rel(got["dk"][cidx, 0], dk_ref[x], floor=1e-2) <= TOL_G, ("dk", int(cidx))
            assert _rel(got["dv"][cidx, 0], dv_ref[x], floor=1e-2) <= TOL_G, ("dv", int(cidx))


def test_whole_tensor_properties(run):
    spec, cu, t = run["spec"], run["cu"], run["t"]
    for name in ("out", "lse", "dq", "dk", "dv"):
        assert bool(torch.isfinite(run[name]).all()), name
    lengths = np.asarray(run["lengths"])
    ones = [j for j in range(len(lengths)) if lengths[j] == 1]
    G = spec.hq // spec.hkv
    for j in ones[:8]:
        r = int(cu[j])
        # a one-token sample returns its V row, has zero dQ / dK, and dV = sum of the group's dO
        v_rep = t["v"][r].float().repeat_interleave(G, dim=0)
        assert torch.equal(run["out"][r].float(), v_rep)
        assert float(run["dq"][r].float().abs().max()) < 1e-5 and float(run["dk"][r].float().abs().max()) < 1e-5
        want = t["dout"][r].float().reshape(spec.hkv, G, -1).sum(1)
        assert float((run["dv"][r].float() - want).abs().max()) <= 0.02 * float(want.abs().max())
    # first row of every sample attends only itself
    firsts = torch.from_numpy(cu[:-1].astype(np.int64)).cuda()
    v_first = t["v"][firsts].float().repeat_interleave(G, dim=1)
    assert torch.equal(run["out"][firsts].float(), v_first)
    lb, plan = run["lb"], run["plan"]
    dq2, dk2, dv2 = lb.libra_attn_pool_bwd(t["q"], t["k"], t["v"], run["out"], run["lse"], t["dout"], plan)
    torch.cuda.synchronize()
    if not run["fused"]:
        # the two-kernel form has no atomics anywhere: the same call again gives bit-identical results
        assert torch.equal(dq2, run["dq"]) and torch.equal(dk2, run["dk"]) and torch.equal(dv2, run["dv"])
    else:
        # the fused form adds into fp32 accumulators in a varying order: equal up to the final bf16 rounding
        for a, b in ((dq2, run["dq"]), (dk2, run["dk"]), (dv2, run["dv"])):
            diff = float((a[:: 7].float() - b[:: 7].float()).abs().max())
            assert diff <= 2.0 ** -7 * float(b[:: 7].float().abs().max())
