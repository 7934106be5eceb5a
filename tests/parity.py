"""Shared helpers of the GPU parity tests (comparison metrics only; no method arithmetic)."""
import numpy as np


def rel_to_max(got, want):
    """max |got - want| / max |want| (the tolerance metric of the benchmark's target)."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    denom = np.abs(want).max()
    return float(np.abs(got - want).max() / (denom if denom > 0 else 1.0))


def band_errors(got, want, cu, band=128):
    """rel_to_max per (sample, `band`-row band): exposes a dropped key block deep inside a
    long sample, where the whole-tensor metric is dominated by the large early rows."""
    worst = 0.0
    for j in range(len(cu) - 1):
        for s in range(int(cu[j]), int(cu[j + 1]), band):
            e = min(s + band, int(cu[j + 1]))
            worst = max(worst, rel_to_max(got[s:e], want[s:e]))
    return worst
