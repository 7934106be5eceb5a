"""Device pool planner (tiles, Algorithm 2, exchange volumes) == oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from oracle import schedule as osched
from paper_2607_23250_b200 import pools

pytestmark = pytest.mark.gpu


def _compare(cu, seq_off, cp, B, H, hq, hkv, d, tau=(3, 100)):
    from paper_2607_23250_b200 import binding as lb
    got = lb.libra_tap_plan(torch.from_numpy(np.asarray(cu, np.int32)).cuda(), seq_off, cp, B, H, hq, hkv, d, *tau)
    L = oracle.tap_layout(cu, seq_off, cp, B, H, hq, hkv, d)
    W = L["n_workers"]
    want = oracle.tap_place(L["f"], L["q_home"], L["v_qo"], L["kv_off"], L["kv_grp"], L["v_g"], L["resident"], W, *tau)
    fwd, bwd = oracle.tap_exchange(cu, seq_off, cp, H, hkv, d, want["sigma"], L["q_home"], L["v_qo"], want["C"],
                                   L["resident"])
    torch.cuda.synchronize()
    assert int(got["status"].item()) == 0
    assert np.array_equal(got["sigma"].cpu().numpy(), want["sigma"])
    assert np.array_equal(got["loads"].cpu().numpy(), want["loads"])
    assert int(got["comm_total"].item()) == want["comm_total"]
    assert np.array_equal(got["fwd_bytes"].cpu().numpy(), fwd)
    assert np.array_equal(got["bwd_bytes"].cpu().numpy(), bwd)
    # the transfer records of the same assignment, and of one that scatters the tiles, equal the oracle's list
    if len(want["sigma"]) <= 4096:
        cu_dev = torch.from_numpy(np.asarray(cu, np.int32)).cuda()
        scattered = np.array([(5 * t + 3) % W for t in range(len(want["sigma"]))], np.int32)
        for sigma in (want["sigma"], scattered):
            rec = lb.libra_tap_schedule(cu_dev, seq_off, torch.from_numpy(sigma).cuda(), cp, B, H, hq, hkv, d)
            assert np.array_equal(rec.cpu().numpy().reshape(-1, 6), osched.schedule(cu, seq_off, cp, B, H, sigma))
    return want, fwd


def test_tiny_hand_checked_layout():
    _compare([0, 5, 6, 16, 20, 32], [0, 16, 32], 2, 4, 2, 4, 2, 8)


@pytest.mark.parametrize("seed", range(12))
def test_random_pools(seed):
    rng = np.random.default_rng(seed)
    P, CP = int(rng.integers(1, 6)), int(rng.choice([1, 2, 4, 8]))
    seqs = [pools.random_layout(rng, int(rng.integers(50, 3000)), int(rng.integers(1, 400))) for _ in range(P)]
    cu = pools.cu_seqlens([x for s in seqs for x in s])
    seq_off = np.concatenate([[0], np.cumsum([sum(s) for s in seqs])]).astype(np.int32)
    H, hkv = [(1, 4), (2, 4), (4, 4), (8, 4), (4, 2)][seed % 5]
    tau = [(3, 100), (0, 1), (50, 100)][seed % 3]
    _compare(cu, seq_off, CP, int(rng.choice([16, 64, 100, 256])), H, 8, hkv, 64, tau)


@pytest.mark.parametrize("P,CP,B,H", [(2, 4, 2048, 2), (8, 2, 1024, 4), (4, 16, 2048, 8)])
def test_long_tailed_pools(P, CP, B, H):
    """Pools of 32768-token sequences of the 30B shape (config 3: Hq 32, Hkv 4, d 128, Pareto-tailed samples)."""
    spec = pools.config(3)
    seqs = [pools.sequence_lengths(spec, i) for i in range(P)]
    cu = pools.cu_seqlens([x for s in seqs for x in s])
    seq_off = np.concatenate([[0], np.cumsum([sum(s) for s in seqs])]).astype(np.int32)
    want, fwd = _compare(cu, seq_off, CP, B, H, spec.hq, spec.hkv, spec.head_dim)
    loads = want["loads"]
    assert loads.max() <= 1.03 * loads.mean() + max(1, oracle.tap_layout(cu, seq_off, CP, B, H, spec.hq, spec.hkv, spec.head_dim)["f"].max())


def test_zero_length_samples_and_short_tail():
    _compare([0, 0, 3, 3, 3, 40, 40, 41], [0, 41], 2, 16, 2, 4, 2, 8)
    _compare([0, 7, 7, 30, 30], [0, 7, 30], 1, 4, 1, 2, 2, 8)


def test_bad_arguments():
    from paper_2607_23250_b200 import binding as lb
    cu = torch.tensor([0, 9], dtype=torch.int32).cuda()
    with pytest.raises(Exception):
        lb.libra_tap_plan(cu, [0, 9], 1, 4, 3, 4, 2, 8)    # 3 shards do not divide 4 heads
    with pytest.raises(Exception):
        lb.libra_tap_plan(cu, [0, 9], 0, 4, 2, 4, 2, 8)
