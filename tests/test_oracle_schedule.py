"""Pins of the exchange-schedule oracle (Section 4.3.3 and the head pieces of Section 4.4): a hand example, the
volumes against the token-by-token exchange matrices (written independently of the record lists), forward =
backward volume, deduplication, W = 1 moves nothing, equal chunk volumes."""
import numpy as np
import pytest

import oracle
from oracle import schedule as osched


def _plan(cu, seq_off, cp, block, H, hq, hkv, d):
    lay = oracle.tap_layout(cu, seq_off, cp, block, H, hq, hkv, d)
    res = oracle.tap_place(lay["f"], lay["q_home"], lay["v_qo"], lay["kv_off"], lay["kv_grp"], lay["v_g"],
                           lay["resident"], lay["n_workers"])
    return lay, res


def test_hand_example():
    # One sequence of 8 tokens on 2 workers (runs [0,4) and [4,8)), blocks of 4, one shard, samples [0,6) and [6,8).
    # Tile 0 = rows 0..3 (home 0), tile 1 = rows 4..7 (home 1).  Put both tiles on worker 0:
    #   tile 1 is away from home: one kind 0 record (rows 4..7 from 1 to 0);
    #   worker 0 needs sample 0 (rows 0..5: run 4..5 lives on worker 1) and sample 1 (rows 6..7, all on worker 1).
    rec = osched.schedule([0, 6, 8], [0, 8], cp=2, block=4, n_shards=1, sigma=[0, 0])
    assert rec.tolist() == [[0, 1, 0, 4, 4, 0], [1, 1, 0, 4, 2, 0], [1, 1, 0, 6, 2, 0]]
    # both tiles at home: worker 0 fetches the rest of sample 0 (rows 4..5) although its tile needs only a causal prefix
    # (a group is fetched whole), worker 1 needs rows 0..3 of sample 0 (its rows 4..5 and sample 1 are local)
    rec = osched.schedule([0, 6, 8], [0, 8], cp=2, block=4, n_shards=1, sigma=[0, 1])
    assert rec.tolist() == [[1, 1, 0, 4, 2, 0], [1, 0, 1, 0, 4, 0]]
    # chunk rule: 8 query heads over 2 kv heads on one shard in 4 chunks: chunks 0, 1 read kv head 0, chunks 2, 3 kv head 1
    heads = [osched.chunk_heads(0, m, 8, 2, 1, 4) for m in range(4)]
    assert [h[0] for h in heads] == [[0, 1], [2, 3], [4, 5], [6, 7]]
    assert [h[1] for h in heads] == [[0], [], [1], []]


@pytest.mark.parametrize("seed", range(6))
def test_volumes_match_the_token_by_token_matrices(seed):
    rng = np.random.default_rng(seed)
    cp = int(rng.choice([1, 2, 4]))
    P = int(rng.choice([1, 2, 3]))
    block = int(rng.choice([4, 8]))
    L = block * cp * int(rng.integers(1, 4))
    seq_off = [L * s for s in range(P + 1)]
    cu = [0]
    for s in range(P):
        left = L
        while left > 0:
            x = int(min(left, rng.integers(1, L + 1)))
            cu.append(cu[-1] + x)
            left -= x
    hkv = int(rng.choice([1, 2]))
    hq = hkv * int(rng.choice([2, 4]))
    H = int(rng.choice([h for h in (1, 2, 4) if hq % h == 0 and (hkv % h == 0 or h % hkv == 0)]))
    d = 8
    lay, res = _plan(cu, seq_off, cp, block, H, hq, hkv, d)
    W = lay["n_workers"]
    fwd, bwd = oracle.tap_exchange(cu, seq_off, cp, H, hkv, d, res["sigma"], lay["q_home"], lay["v_qo"], res["C"],
                                   lay["resident"])
    rec = osched.schedule(cu, seq_off, cp, block, H, res["sigma"])
    width = hq // H
    for M in [m for m in (1, 2, 4) if width % m == 0]:
        f_sum = np.zeros((W, W), np.int64)
        b_sum = np.zeros((W, W), np.int64)
        per_chunk = []
        for m in range(M):
            f, b = osched.chunk_bytes(rec, m, hq, hkv, d, H, M, W)
            f_sum += f
            b_sum += b
            per_chunk.append((f, b))
        assert np.array_equal(f_sum, fwd) and np.array_equal(b_sum, bwd)        # the chunks add up to the whole exchange
        assert f_sum.sum() == b_sum.sum()                                       # backward volume = forward volume
        kvps = hkv // H if H <= hkv else 1
        if kvps % M == 0:                                                       # every chunk then moves the same bytes
            for f, b in per_chunk[1:]:
                assert np.array_equal(f, per_chunk[0][0]) and np.array_equal(b, per_chunk[0][1])
    # deduplication: one fetch per (destination, sample rows, shard, source)
    kv = [tuple(r) for r in rec.tolist() if r[0] == 1]
    assert len(kv) == len(set(kv))
    assert all(r[1] != r[2] for r in rec.tolist())                              # nothing is sent to oneself
    if W == 1:
        assert len(rec) == 0


def test_every_tile_at_home_moves_only_kv():
    cu, seq_off = [0, 5, 16, 32], [0, 16, 32]
    lay = oracle.tap_layout(cu, seq_off, 2, 4, 2, 4, 2, 8)
    rec = osched.schedule(cu, seq_off, 2, 4, 2, lay["q_home"])
    assert (rec[:, 0] == 1).all()
    # a sample wholly inside one worker's run is never fetched by that worker
    for kind, src, dst, tok0, ntok, shard in rec.tolist():
        assert src != dst and ntok > 0
