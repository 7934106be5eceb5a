"""Device VRSP (Algorithm 1) == oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_23250_b200 import pools

pytestmark = pytest.mark.gpu


def _compare(work_np, P):
    from paper_2607_23250_b200 import binding as lb
    got = lb.libra_vrsp_place(torch.from_numpy(work_np).cuda(), P)
    want = oracle.vrsp_place(work_np, P)
    torch.cuda.synchronize()
    for k in ("order", "pool_of_seq", "pool_load"):
        assert np.array_equal(got[k].cpu().numpy(), want[k]), k


def test_hand_example():
    _compare(np.array([9, 7, 6, 5, 4, 1], dtype=np.int64), 2)


@pytest.mark.parametrize("seed", range(12))
def test_random_windows(seed):
    rng = np.random.default_rng(seed)
    P = int(rng.choice([1, 2, 3, 8, 16, 64]))
    K = int(rng.choice([1, 2, 31, 32, 33, 100, 128, 129, 700, 1024]))
    hi = 20 if seed % 3 == 0 else 10**13          # many equal works and equal loads / none
    _compare(rng.integers(0, hi, size=P * K).astype(np.int64), P)


@pytest.mark.parametrize("P", [1, 4, 8, 32, 128])
def test_long_tailed_window(P):
    spec = pools.config(3, 0.0, 7)
    lengths = [pools.sequence_lengths(spec, i) for i in range(128)]
    offs = np.concatenate([[0], np.cumsum([x for s in lengths for x in s])]).astype(np.int32)
    first = np.concatenate([[0], np.cumsum([len(s) for s in lengths])]).astype(np.int32)
    from paper_2607_23250_b200 import binding as lb
    work = lb.libra_vrsp_work(torch.from_numpy(offs).cuda(), torch.from_numpy(first).cuda())
    want = oracle.vrsp_work(offs, first)
    assert np.array_equal(work.cpu().numpy(), want)
    _compare(want, P)


def test_bad_arguments():
    from paper_2607_23250_b200 import binding as lb
    w = torch.arange(6, dtype=torch.int64).cuda()
    with pytest.raises(Exception):
        lb.libra_vrsp_place(w, 4)      # P does not divide D
    with pytest.raises(Exception):
        lb.libra_vrsp_place(w, 0)
