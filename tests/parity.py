"""Shared helpers of the GPU parity tests (comparison metrics only; no method arithmetic)."""
import numpy as np


def rel_to_max(got, want):
    """max |got - want| / max |want| (the tolerance metric of the benchmark's target)."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    denom = np.abs(want).max()
    return float(np.abs(got - want).max() / (denom if denom > 0 else 1.0))


def band_errors(got, want, cu, band=128, floor=0.05):
    """Max-abs error per (sample, `band`-row band) relative to that band's own max magnitude
    (floored at `floor` x the tensor's max so that all-zero bands, e.g. dQ of one-token
    samples, do not divide by nothing).  Exposes a dropped key block deep inside a long
    sample, where the whole-tensor metric is dominated by the large early rows."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    gmax = float(np.abs(want).max()) or 1.0
    worst = 0.0
    for j in range(len(cu) - 1):
        if int(cu[j + 1]) - int(cu[j]) < 2 * band:
            continue  # short samples: few keys per row, the whole-tensor metric already resolves them
        for s in range(int(cu[j]), int(cu[j + 1]), band):
            e = min(s + band, int(cu[j + 1]))
            denom = max(float(np.abs(want[s:e]).max()), floor * gmax)
            worst = max(worst, float(np.abs(got[s:e] - want[s:e]).max()) / denom)
    return worst
