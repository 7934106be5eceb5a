"""Device tile plan == oracle plan, bit for bit (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools

pytestmark = pytest.mark.gpu

KEYS = ("weight", "order", "cta_of_tile", "cta_offsets", "cta_tiles", "loads")


def _compare(cu_np, H, tile, W, tile_kv=0, H_kv=0):
    from paper_2607_23250_b200 import binding as lb
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, H, tile, n_workers=W, tile_kv=tile_kv, n_heads_kv=H_kv)
    assert plan.status() == 0
    for direction, d_or, t, h in ((lb.LIBRA_DIR_Q, 0, tile, H), (lb.LIBRA_DIR_KV, 1, tile_kv or 128, H_kv or H)):
        got = plan.export(direction)
        want = oracle.plan(cu_np, h, t, W, d_or)
        assert got["n_blocks"] == want["n_blocks"]
        for k in KEYS:
            assert np.array_equal(got[k], want[k]), (direction, k)
    plan.destroy()


def test_hand_example():
    _compare(np.array([0, 5, 6, 16], dtype=np.int32), 1, 4, 2, tile_kv=4)


@pytest.mark.parametrize("seed", range(10))
def test_random_tiny_layouts(seed):
    rng = np.random.default_rng(seed)
    lengths = pools.random_layout(rng, int(rng.integers(10, 5000)), int(rng.integers(1, 700)))
    _compare(pools.cu_seqlens(lengths), int(rng.integers(1, 9)), int(rng.choice([1, 3, 16, 100, 128, 256])),
             int(rng.integers(1, 400)), tile_kv=int(rng.choice([7, 64, 128])), H_kv=int(rng.integers(1, 5)))


@pytest.mark.parametrize("idx,skew", [(1, 0), (2, 0), (3, 0), (4, 0), (5, 0), (5, 0.25), (5, 0.5), (5, 1.0)])
def test_benchmark_configs(idx, skew):
    spec = pools.config(idx, skew)
    cu = pools.cu_seqlens(pools.pool_lengths(spec))
    _compare(cu, spec.hq, 256, 148, tile_kv=128, H_kv=spec.hkv)


def _compare_blocks(cu_np, H, tile, W, tile_kv, H_kv, g, uq, ukv):
    """Block-count weight model: device plan == oracle plan, bit for bit."""
    from paper_2607_23250_b200 import binding as lb
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, H, tile, n_workers=W, tile_kv=tile_kv, n_heads_kv=H_kv,
                               weight_model=lb.LIBRA_WEIGHT_BLOCKS, cost_block=g, unit_cost_q=uq, unit_cost_kv=ukv)
    assert plan.status() == 0
    for direction, d_or, t, h, u in ((lb.LIBRA_DIR_Q, 0, tile, H, uq), (lb.LIBRA_DIR_KV, 1, tile_kv, H_kv, ukv)):
        got = plan.export(direction)
        want = oracle.plan(cu_np, h, t, W, d_or, weight_model=1, cost_block=g or 128, unit_cost=u)
        for k in KEYS:
            assert np.array_equal(got[k], want[k]), (direction, k)
    plan.destroy()


@pytest.mark.parametrize("seed", range(8))
def test_block_model_random_layouts(seed):
    rng = np.random.default_rng(300 + seed)
    lengths = pools.random_layout(rng, int(rng.integers(10, 6000)), int(rng.integers(1, 700)))
    _compare_blocks(pools.cu_seqlens(lengths), int(rng.integers(1, 9)), int(rng.choice([3, 16, 100, 128, 256])),
                    int(rng.integers(1, 400)), int(rng.choice([7, 64, 128])), int(rng.integers(1, 5)),
                    int(rng.choice([0, 4, 32, 128])), int(rng.integers(0, 30)), int(rng.integers(0, 30)))


@pytest.mark.parametrize("idx,skew", [(1, 0), (2, 0), (3, 0), (5, 0.5)])
def test_block_model_benchmark_configs(idx, skew):
    spec = pools.config(idx, skew)
    cu = pools.cu_seqlens(pools.pool_lengths(spec))
    _compare_blocks(cu, spec.hkv, 256, 148, 128, spec.hkv, 0, 12, 6)


def test_block_model_rejects_bad_options():
    from paper_2607_23250_b200 import binding as lb
    cu = torch.tensor([0, 9], dtype=torch.int32).cuda()
    for kw in (dict(weight_model=2), dict(weight_model=1, cost_block=-1), dict(weight_model=1, unit_cost_q=-3)):
        with pytest.raises(Exception):
            lb.libra_plan_tiles(cu, 1, 4, n_workers=2, **kw)


def test_edge_cases():
    _compare(np.array([0, 1], dtype=np.int32), 1, 256, 148)                      # one token
    _compare(np.array([0, 0, 3, 3, 3, 700, 700], dtype=np.int32), 2, 256, 5)     # empty samples, ragged tail
    _compare(np.arange(0, 1001, dtype=np.int32), 3, 128, 1000)                   # all length-1, W > tiles/..
    _compare(np.array([0, 65536], dtype=np.int32), 4, 256, 148)                  # equal-weight ties across shards


def test_bad_cu_seqlens_is_reported_not_crashing():
    from paper_2607_23250_b200 import binding as lb
    for bad in ([1, 5, 9], [0, 7, 5, 9]):
        cu = torch.tensor(bad, dtype=torch.int32).cuda()
        plan = lb.libra_plan_tiles(cu, 1, 4, n_workers=2, total_tokens=9)
        assert plan.status() == lb.ERR_BAD_SEQLENS
        plan.destroy()
    with pytest.raises(lb.LibraError):
        lb.libra_plan_tiles(torch.tensor([0, 4], dtype=torch.int32).cuda(), 0, 4)


# ---- pair tiles (key block x query chunk x head): the fused backward's units ---------------------------------

def _compare_pairs(cu_np, H_kv, tile_kv, chunk, W):
    from paper_2607_23250_b200 import binding as lb
    cu = torch.from_numpy(cu_np).cuda()
    plan = lb.libra_plan_tiles(cu, H_kv, 256, n_workers=W, directions=lb.LIBRA_DIR_PAIR, tile_kv=tile_kv, n_heads_kv=H_kv,
                               pair_chunk=chunk)
    assert plan.status() == 0
    kb, qc, chunk_used = plan.export_pairs()
    want = oracle.plan_pairs(cu_np, H_kv, tile_kv, chunk_used, W)       # the planner may have widened the chunk
    got = plan.export(lb.LIBRA_DIR_PAIR)
    assert got["n_blocks"] == want["n_blocks"] <= 262144
    assert np.array_equal(kb, want["key_block"]) and np.array_equal(qc, want["query_chunk"])
    for k in KEYS:
        assert np.array_equal(got[k], want[k]), k
    plan.destroy()
    return chunk_used


def test_pair_tiles_hand_example():
    _compare_pairs(np.array([0, 5, 6, 16], dtype=np.int32), 1, 4, 8, 2)


@pytest.mark.parametrize("seed", range(8))
def test_pair_tiles_random_layouts(seed):
    rng = np.random.default_rng(100 + seed)
    lengths = pools.random_layout(rng, int(rng.integers(10, 4000)), int(rng.integers(1, 900)))
    tile = int(rng.choice([4, 16, 128]))
    _compare_pairs(pools.cu_seqlens(lengths), int(rng.integers(1, 5)), tile, tile * int(rng.choice([1, 2, 8])),
                   int(rng.integers(1, 300)))


@pytest.mark.parametrize("idx,skew", [(1, 0), (2, 0), (3, 0)])
def test_pair_tiles_benchmark_configs(idx, skew):
    spec = pools.config(idx, skew)
    cu = pools.cu_seqlens(pools.pool_lengths(spec))
    _compare_pairs(cu, spec.hkv, 128, 2048, 148)


def test_pair_chunk_is_widened_until_the_pair_blocks_fit():
    # a 60000-token sample at 16-token blocks and chunks would have about 7 million pair-blocks
    cu = np.array([0, 60000], dtype=np.int32)
    assert _compare_pairs(cu, 1, 16, 16, 7) > 16
