"""Pins for the oracle of Algorithm 2 (communication-aware placement), its pool tables and exchange volumes:
a hand-evaluated instance, an independent set-based re-implementation, reduction to the single-GPU plan
when nothing costs communication, brute-force tables, and the forward = backward volume statement."""
import os

import numpy as np
import pytest

import oracle
from paper_2607_23250_b200 import pools

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, *vals = line.split()
                out[key] = [int(x) for x in vals]
    return out


def test_hand_example():
    g = _golden("tap_hand_example.txt")
    r = oracle.tap_place(g["work"], g["q_home"], g["v_qo"], g["kv_off"], g["kv_grp"], g["v_g"], g["resident"],
                         g["workers"][0])
    assert r["sigma"].tolist() == g["sigma"]
    assert r["loads"].tolist() == g["loads"]
    assert r["comm_total"] == g["comm_total"][0]


def _sets_tap(f, q_home, v_qo, K, v_g, resident, W, tau=(3, 100)):
    """Algorithm 2 with Python sets and tuple keys; exact rational cap via integers."""
    order = sorted(range(len(f)), key=lambda t: (-f[t], t))
    L = [0] * W
    C = [{g for g in range(len(v_g)) if resident[g] == r} for r in range(W)]
    total = sum(f)
    sigma = [None] * len(f)
    comm = 0
    for t in order:
        def delta(r):
            return sum(v_g[g] for g in K[t] - C[r]) + (v_qo[t] if r != q_home[t] else 0)
        F = [r for r in range(W) if tau[1] * W * (L[r] + f[t]) <= (tau[1] + tau[0]) * total]
        r = min(F, key=lambda r: (delta(r), L[r], r)) if F else min(range(W), key=lambda r: (L[r], delta(r), r))
        comm += delta(r)
        sigma[t] = r; L[r] += f[t]; C[r] |= K[t]
    return sigma, L, C, comm


@pytest.mark.parametrize("seed", range(12))
def test_against_set_based_reimplementation(seed):
    rng = np.random.default_rng(seed)
    NT, W, NG = int(rng.integers(1, 60)), int(rng.integers(1, 9)), int(rng.integers(1, 12))
    f = rng.integers(0, 30, NT).tolist()
    q_home = rng.integers(0, W, NT).tolist()
    v_qo = (2 * rng.integers(0, 6, NT)).tolist()
    K = [set(rng.choice(NG, size=int(rng.integers(0, min(NG, 4) + 1)), replace=False).tolist()) for _ in range(NT)]
    v_g = rng.integers(0, 20, NG).tolist()
    resident = rng.integers(-1, W, NG).tolist()
    kv_off = np.concatenate([[0], np.cumsum([len(k) for k in K])])
    kv_grp = [g for k in K for g in sorted(k)]
    r = oracle.tap_place(f, q_home, v_qo, kv_off, kv_grp, v_g, resident, W)
    sigma, L, C, comm = _sets_tap(f, q_home, v_qo, K, v_g, resident, W)
    assert r["sigma"].tolist() == sigma
    assert r["loads"].tolist() == L
    assert r["comm_total"] == comm
    assert [set(np.nonzero(r["C"][w])[0].tolist()) for w in range(W)] == C


@pytest.mark.parametrize("W", [1, 2, 7, 148])
def test_without_communication_it_is_the_single_gpu_plan(W):
    """With every volume zero both branches of Algorithm 2 pick the least-loaded, lowest-index worker."""
    lengths = pools.pool_lengths(pools.config(1))
    p = oracle.plan(pools.cu_seqlens(lengths), 4, 128, W, 0)
    NT = len(p["weight"])
    r = oracle.tap_place(p["weight"], [0] * NT, [0] * NT, list(range(NT + 1)), [0] * NT, [0], [-1], W)
    assert r["sigma"].tolist() == p["cta_of_tile"].tolist()
    assert r["loads"].tolist() == p["loads"].tolist()
    assert r["comm_total"] == 0


def _layout_case(seed):
    rng = np.random.default_rng(seed)
    P, CP = int(rng.integers(1, 4)), int(rng.choice([1, 2, 4]))
    seqs = [pools.random_layout(rng, int(rng.integers(8, 120)), int(rng.integers(1, 40))) for _ in range(P)]
    cu = pools.cu_seqlens([x for s in seqs for x in s])
    seq_off = np.concatenate([[0], np.cumsum([sum(s) for s in seqs])]).astype(np.int32)
    H, hkv = (2, 4) if seed % 2 else (4, 2)
    return cu, seq_off, P, CP, int(rng.choice([4, 8, 16])), H, 8, hkv, 16


@pytest.mark.parametrize("seed", range(8))
def test_layout_tables_brute_force(seed):
    cu, seq_off, P, CP, B, H, hq, hkv, d = _layout_case(seed)
    L = oracle.tap_layout(cu, seq_off, CP, B, H, hq, hkv, d)
    n = len(cu) - 1
    sid = np.repeat(np.arange(n), np.diff(cu))
    owner = np.empty(cu[-1], np.int64)
    for s in range(P):
        ln = seq_off[s + 1] - seq_off[s]; run = -(-ln // CP)
        owner[seq_off[s]:seq_off[s + 1]] = s * CP + np.arange(ln) // run
    t = 0
    for s in range(P):
        for q0 in range(seq_off[s], seq_off[s + 1], B):
            q1 = min(q0 + B, seq_off[s + 1])
            pairs = sum(int(p - cu[sid[p]] + 1) for p in range(q0, q1))
            for h in range(H):
                assert L["f"][t] == pairs
                assert L["q_home"][t] == owner[q0]
                assert L["v_qo"][t] == 2 * (q1 - q0) * (hq // H) * d * 2
                assert L["kv_grp"][L["kv_off"][t]:L["kv_off"][t + 1]].tolist() == [j * H + h for j in sorted(set(sid[q0:q1]))]
                t += 1
    assert t == len(L["f"])
    kvps = hkv // H if H <= hkv else 1
    for j in range(n):
        own = set(owner[cu[j]:cu[j + 1]].tolist())
        res = next(iter(own)) if len(own) == 1 else -1
        for h in range(H):
            assert L["v_g"][j * H + h] == 2 * (cu[j + 1] - cu[j]) * kvps * d * 2
            assert L["resident"][j * H + h] == res
    # a one-sequence pool on one worker: f is the single-GPU plan's weight
    if P == 1:
        assert L["f"].tolist() == oracle.plan(cu, H, B, 3, 0)["weight"].tolist()


@pytest.mark.parametrize("seed", range(8))
def test_exchange_volumes(seed):
    cu, seq_off, P, CP, B, H, hq, hkv, d = _layout_case(100 + seed)
    L = oracle.tap_layout(cu, seq_off, CP, B, H, hq, hkv, d)
    W = P * CP
    r = oracle.tap_place(L["f"], L["q_home"], L["v_qo"], L["kv_off"], L["kv_grp"], L["v_g"], L["resident"], W)
    fwd, bwd = oracle.tap_exchange(cu, seq_off, CP, H, hkv, d, r["sigma"], L["q_home"], L["v_qo"], r["C"], L["resident"])
    assert fwd.sum() == bwd.sum()                                  # Section 4.3.3: equal volume, reversed paths
    assert np.array_equal(np.diag(fwd), np.zeros(W, np.int64))     # nothing is sent to oneself
    # independent recomputation: Q/O part symmetric, KV part from owners to destinations
    n = len(cu) - 1
    owner = np.empty(cu[-1], np.int64)
    for s in range(P):
        ln = seq_off[s + 1] - seq_off[s]; run = -(-ln // CP)
        owner[seq_off[s]:seq_off[s + 1]] = s * CP + np.arange(ln) // run
    kvps = hkv // H if H <= hkv else 1
    want = np.zeros((W, W), np.int64)
    for t, (q, dst) in enumerate(zip(L["q_home"], r["sigma"])):
        if q != dst:
            want[q, dst] += L["v_qo"][t] // 2; want[dst, q] += L["v_qo"][t] // 2
    used = [set() for _ in range(W)]
    for t, dst in enumerate(r["sigma"]):
        used[dst] |= set(L["kv_grp"][L["kv_off"][t]:L["kv_off"][t + 1]].tolist())
    kv = np.zeros((W, W), np.int64)
    for dst in range(W):
        for g in used[dst]:
            j = g // H
            for tok in range(cu[j], cu[j + 1]):
                if owner[tok] != dst:
                    kv[owner[tok], dst] += 2 * kvps * d * 2
    assert np.array_equal(fwd, want + kv)
    assert np.array_equal(bwd, want + kv.T)
    assert r["loads"].sum() == L["f"].sum() and ((0 <= r["sigma"]) & (r["sigma"] < W)).all()
    if W == 1:
        assert fwd.sum() == 0
