"""Pins for the plan oracle: hand-evaluated example, closed forms, brute force, invariants.

None of these retypes the oracle's own loops: weights are checked against brute-force
pair enumeration over a dense mask, against closed forms, and against totals; placement
is checked against an independent event simulation (a heap), Graham's bound and
conservation laws.
"""
import heapq
import os

import numpy as np
import pytest

import oracle
from paper_2607_23250_b200 import pools

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [int(x) for x in vals]
    return out


def test_hand_example():
    g = _read_golden("plan_hand_example.txt")
    cu = np.array(g["cu_seqlens"], dtype=np.int32)
    p = oracle.plan(cu, g["heads"][0], g["tile"][0], g["workers"][0], direction=0)
    assert p["weight"].tolist() == g["weight_q"]
    assert p["order"].tolist() == g["order_q"]
    assert p["cta_of_tile"].tolist() == g["cta_of_tile_q"]
    assert p["loads"].tolist() == g["loads_q"]
    assert p["cta_offsets"].tolist() == [0, 1, 4]
    assert p["cta_tiles"].tolist() == [3, 2, 0, 1]
    pk = oracle.plan(cu, g["heads"][0], g["tile"][0], g["workers"][0], direction=1)
    assert pk["weight"].tolist() == g["weight_kv"]


def test_paper_long_sample_statement():
    g = _read_golden("paper_statements.txt")
    big, small, cnt = g["long_sample_tokens"][0], g["short_sample_tokens"][0], g["short_sample_count"][0]
    # one block spanning everything: weight = causal pairs of the layout
    w_big = oracle.plan(pools.cu_seqlens([big]), 1, big, 1)["weight"][0]
    w_small = oracle.plan(pools.cu_seqlens([small] * cnt), 1, big, 1)["weight"][0]
    ratio = w_big / w_small
    # pairs are l(l+1)/2, the proxy is l^2: the ratio is 10 up to the +l term
    assert abs(ratio - g["flops_ratio"][0]) < 0.01


def _brute_weights(lengths, tile, direction):
    """Dense mask enumeration: count (q, k) pairs with same sample and k <= q, per block."""
    T = sum(lengths)
    sid = np.repeat(np.arange(len(lengths)), lengths)
    pos = np.arange(T)
    mask = (sid[:, None] == sid[None, :]) & (pos[None, :] <= pos[:, None])  # [q, k]
    nb = -(-T // tile)
    per_token = mask.sum(axis=1) if direction == 0 else mask.sum(axis=0)
    return [int(per_token[b * tile:(b + 1) * tile].sum()) for b in range(nb)]


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("direction", [0, 1])
def test_weights_brute_force(seed, direction):
    rng = np.random.default_rng(seed)
    total = int(rng.integers(20, 300))
    lengths = pools.random_layout(rng, total, int(rng.integers(1, 90)))
    tile = int(rng.choice([1, 3, 4, 7, 16, 32, 64]))
    H = int(rng.integers(1, 4))
    p = oracle.plan(pools.cu_seqlens(lengths), H, tile, 5, direction)
    want = _brute_weights(lengths, tile, direction)
    assert p["n_blocks"] == len(want)
    assert p["weight"].reshape(-1, H).tolist() == [[w] * H for w in want]


def test_weights_closed_form_single_sample():
    # one sample of length l cut at B: block b holds local rows bB..bB+B-1, each with row+1 keys
    l, B = 4096, 128
    p = oracle.plan(pools.cu_seqlens([l]), 1, B, 7, 0)
    b = np.arange(l // B, dtype=np.int64)
    assert p["weight"].tolist() == (B * (2 * b * B + B + 1) // 2).tolist()
    # key-major is the mirror image
    pk = oracle.plan(pools.cu_seqlens([l]), 1, B, 7, 1)
    assert pk["weight"].tolist() == p["weight"][::-1].tolist()


@pytest.mark.parametrize("idx,skew", [(1, 0), (2, 0), (3, 0), (5, 0.5)])
def test_weight_totals_on_configs(idx, skew):
    spec = pools.config(idx, skew)
    lengths = np.array(pools.pool_lengths(spec), dtype=np.int64)
    pairs = int((lengths * (lengths + 1) // 2).sum())
    H = spec.hkv
    for direction in (0, 1):
        p = oracle.plan(pools.cu_seqlens(lengths), H, 128, 148, direction)
        assert int(p["weight"].sum()) == H * pairs
        assert int(p["loads"].sum()) == H * pairs


def _heap_lpt(weight, W):
    """Independent placement: event simulation with a heap of (load, worker)."""
    order = sorted(range(len(weight)), key=lambda t: (-int(weight[t]), t))
    heap = [(0, r) for r in range(W)]
    heapq.heapify(heap)
    cta = [0] * len(weight)
    lists = [[] for _ in range(W)]
    for t in order:
        load, r = heapq.heappop(heap)
        cta[t] = r
        lists[r].append(t)
        heapq.heappush(heap, (load + int(weight[t]), r))
    loads = [0] * W
    for t, r in enumerate(cta):
        loads[r] += int(weight[t])
    return order, cta, lists, loads


@pytest.mark.parametrize("seed", range(8))
def test_placement_vs_heap_simulation(seed):
    rng = np.random.default_rng(100 + seed)
    lengths = pools.random_layout(rng, int(rng.integers(50, 2000)), int(rng.integers(1, 400)))
    tile = int(rng.choice([4, 16, 32, 128]))
    H = int(rng.integers(1, 5))
    W = int(rng.integers(1, 12))
    p = oracle.plan(pools.cu_seqlens(lengths), H, tile, W, int(seed % 2))
    order, cta, lists, loads = _heap_lpt(p["weight"], W)
    assert p["order"].tolist() == order
    assert p["cta_of_tile"].tolist() == cta
    assert p["loads"].tolist() == loads
    off = p["cta_offsets"]
    for r in range(W):
        assert p["cta_tiles"][off[r]:off[r + 1]].tolist() == lists[r]


@pytest.mark.parametrize("idx,skew,W", [(2, 0, 148), (3, 0, 148), (5, 1.0, 296)])
def test_placement_invariants(idx, skew, W):
    spec = pools.config(idx, skew)
    cu = pools.cu_seqlens(pools.pool_lengths(spec))
    p = oracle.plan(cu, spec.hkv, 128, W, 0)
    nt = p["weight"].size
    # every tile exactly once
    assert sorted(p["cta_tiles"].tolist()) == list(range(nt))
    assert p["cta_offsets"][0] == 0 and p["cta_offsets"][-1] == nt
    # loads are the sums of the assigned weights
    loads = np.zeros(W, dtype=np.int64)
    np.add.at(loads, p["cta_of_tile"], p["weight"])
    assert loads.tolist() == p["loads"].tolist()
    # list scheduling bounds: spread at most one tile; Graham's bound
    wmax = int(p["weight"].max())
    assert int(loads.max() - loads.min()) <= wmax
    assert loads.max() <= loads.mean() + wmax * (1 - 1 / W) + 1e-9
    # order is by decreasing weight then id
    o = p["order"]
    w = p["weight"][o]
    assert np.all((w[:-1] > w[1:]) | ((w[:-1] == w[1:]) & (o[:-1] < o[1:])))


def test_zero_length_samples_and_ragged_tail():
    # repeated offsets (empty samples) contribute nothing; last block short
    cu = np.array([0, 0, 5, 5, 6, 16, 16, 19], dtype=np.int32)
    a = oracle.plan(cu, 2, 4, 3, 0)
    b = oracle.plan(np.array([0, 5, 6, 16, 19], dtype=np.int32), 2, 4, 3, 0)
    for key in ("weight", "order", "cta_of_tile", "cta_tiles", "loads"):
        assert a[key].tolist() == b[key].tolist()
    assert a["n_blocks"] == 5
    assert a["weight"].reshape(-1, 2)[-1, 0] == 1 + 2 + 3  # tokens 16..18 of the last sample


# ---- block-count weight (a time proxy, not in the paper) -------------------------------------------

def _brute_block_weights(lengths, tile, direction, g, unit_cost):
    """Every visible (q, k) pair marks the cell (q // g, k // g); a tile's weight counts, per chunk piece
    it holds, the marked cells of that piece's rows (query-major) or columns (key-major)."""
    T = sum(lengths)
    sid = np.repeat(np.arange(len(lengths)), lengths)
    cells = {}  # piece -> set of chunks on the other axis
    for q in range(T):
        for k in range(q + 1):
            if sid[q] != sid[k]:
                continue
            own, other = (q, k) if direction == 0 else (k, q)
            cells.setdefault((own // tile, own // g), set()).add(other // g)
    nb = -(-T // tile)
    w = [0] * nb
    for (b, _chunk), others in cells.items():
        w[b] += 8 * len(others) + unit_cost
    return w


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("direction", [0, 1])
def test_block_weights_brute_force(seed, direction):
    rng = np.random.default_rng(100 + seed)
    total = int(rng.integers(20, 260))
    lengths = [x for x in pools.random_layout(rng, total, int(rng.integers(1, 90)))]
    g = int(rng.choice([2, 4, 8, 16]))
    tile = int(rng.choice([g, 2 * g, 3 * g, 5, 7, 1]))   # aligned, and tiles that cut chunks into pieces
    unit = int(rng.integers(0, 20))
    H = int(rng.integers(1, 4))
    p = oracle.plan(pools.cu_seqlens(lengths), H, tile, 5, direction, weight_model=1, cost_block=g, unit_cost=unit)
    want = _brute_block_weights(lengths, tile, direction, g, unit)
    assert p["weight"].reshape(-1, H).tolist() == [[w] * H for w in want]


def test_block_weights_single_sample_closed_form():
    # one sample of 10 chunks, tile = 2 chunks: row chunk i sees chunks 0..i, key chunk i is seen by chunks i..9
    g, n = 16, 10
    pq = oracle.plan(pools.cu_seqlens([g * n]), 1, 2 * g, 3, 0, weight_model=1, cost_block=g, unit_cost=5)
    pk = oracle.plan(pools.cu_seqlens([g * n]), 1, 2 * g, 3, 1, weight_model=1, cost_block=g, unit_cost=5)
    assert pq["weight"].tolist() == [8 * ((2 * b + 1) + (2 * b + 2)) + 10 for b in range(5)]
    assert pk["weight"].tolist() == [8 * ((n - 2 * b) + (n - 2 * b - 1)) + 10 for b in range(5)]
    assert pq["weight"].sum() == pk["weight"].sum()   # both count the same lower-triangular cells


@pytest.mark.parametrize("seed", range(4))
def test_block_model_placement_vs_heap_simulation(seed):
    rng = np.random.default_rng(200 + seed)
    lengths = pools.random_layout(rng, int(rng.integers(500, 4000)), int(rng.integers(1, 900)))
    H, W = int(rng.integers(1, 5)), int(rng.integers(2, 40))
    p = oracle.plan(pools.cu_seqlens(lengths), H, 256, W, 0, weight_model=1, cost_block=128, unit_cost=12)
    order, owner, _lists, loads = _heap_lpt(p["weight"], W)
    assert p["order"].tolist() == order
    assert p["cta_of_tile"].tolist() == owner
    assert p["loads"].tolist() == loads


# ---- pair tiles (key block x query chunk x head): the fused backward's units ---------------------------------

def _visible_pairs(cu):
    """All (query, key) pairs of the pool: same sample, key position <= query position."""
    out = []
    for j in range(len(cu) - 1):
        for q in range(cu[j], cu[j + 1]):
            for k in range(cu[j], q + 1):
                out.append((q, k))
    return out


@pytest.mark.parametrize("cu,tile,chunk", [([0, 5, 6, 16], 4, 8), ([0, 3, 3, 20, 21, 37], 4, 4), ([0, 40], 8, 16),
                                           ([0, 1, 2, 3, 30], 4, 12), ([0, 9, 33], 16, 16), ([0, 70], 4, 16)])
def test_pair_tiles_are_the_live_cells_of_the_score_matrix(cu, tile, chunk):
    H, W = 2, 3
    res = oracle.plan_pairs(cu, H, tile, chunk, W)
    nu = res["n_blocks"]
    # brute force over every visible pair: the live cells, grouped by (query chunk, key block)
    cells = {(q // tile, k // tile) for q, k in _visible_pairs(cu)}
    groups = {}
    for i, j in cells:
        groups[(i * tile // chunk, j)] = groups.get((i * tile // chunk, j), 0) + 1
    listed = list(zip(res["query_chunk"].tolist(), res["key_block"].tolist()))
    assert listed == sorted(groups)                                  # chunk by chunk, key blocks ascending
    for u, cell in enumerate(listed):
        for h in range(H):
            assert res["weight"][h * nu + u] == groups[cell]          # head-major ids, the same weight for every head
    assert int(res["weight"].sum()) == H * len(cells)
    # placement: in tile-id order, least-loaded worker, lowest index on ties
    assert res["order"].tolist() == list(range(nu * H))
    loads, lists = [0] * W, [[] for _ in range(W)]
    for t in range(nu * H):
        r = min(range(W), key=lambda x: (loads[x], x))
        assert res["cta_of_tile"][t] == r
        loads[r] += int(res["weight"][t])
        lists[r].append(t)
    assert res["loads"].tolist() == loads
    assert res["cta_tiles"].tolist() == [t for l in lists for t in l]
    assert max(loads) - min(loads) <= int(res["weight"].max())     # list scheduling: no worker is a whole tile ahead


def test_pair_tiles_of_one_long_sample_in_closed_form():
    """One sample of n row blocks, chunks of R blocks: key block j meets chunk c in min(n, (c+1)R) - max(j, cR) cells."""
    tile, R, n = 8, 4, 11
    res = oracle.plan_pairs([0, n * tile], 1, tile, R * tile, 5)
    want = [(c, j, min(n, (c + 1) * R) - max(j, c * R)) for c in range((n + R - 1) // R) for j in range(min(n, (c + 1) * R))]
    got = list(zip(res["query_chunk"].tolist(), res["key_block"].tolist(), res["weight"].tolist()))
    assert got == want
