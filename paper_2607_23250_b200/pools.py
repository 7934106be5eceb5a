"""Seeded synthetic attention pools (input generators only).

A *pool* is a set of packed sequences laid end to end on one token axis; each
packed sequence is a concatenation of samples whose lengths follow a long-tailed
distribution (median 644 tokens, tail reaching the sequence length), which is the
shape of the corpus the paper describes in its motivation section (sample-length
figure, Section 3.1) with the attention-layer head shapes of its Table 1.

This module draws sample lengths and random tensors.  It contains none of the
method's arithmetic (no tile weights, no attention, no FLOP formulas) so that the
CPU oracle and the CUDA library can both be fed from it without sharing code.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

MEDIAN_LEN = 644.0
SIGMA = 1.6
_DRAW = 4096  # log-normal lengths are drawn in batches of this size


@dataclass(frozen=True)
class PoolSpec:
    """Shape of one synthetic pool (one attention layer's worth of input)."""
    name: str
    config_index: int          # position in the benchmark's config list (1-based)
    n_seqs: int                # packed sequences in the pool
    seq_len: int               # tokens per packed sequence (L)
    hq: int
    hkv: int
    head_dim: int
    big: str = "none"          # "none" | "pareto" | "fixed" | "frac"
    big_len: int = 0           # for "fixed"
    big_frac: float = 0.0      # for "frac": one sample of big_frac * L per sequence
    seed: int = 0

    @property
    def total_tokens(self) -> int:
        return self.n_seqs * self.seq_len


def _lognormal_fill(rng: np.random.Generator, target: int, L: int) -> list[int]:
    """Log-normal(median 644, sigma 1.6) lengths, rounded, clipped to [1, L],
    consumed in draw order until they sum to `target`; the last one is cut short."""
    out: list[int] = []
    filled = 0
    while filled < target:
        batch = np.clip(np.rint(np.exp(rng.normal(math.log(MEDIAN_LEN), SIGMA, size=_DRAW))), 1, L)
        for x in batch.astype(np.int64):
            x = int(min(x, target - filled))
            out.append(x)
            filled += x
            if filled >= target:
                break
    return out


def sequence_lengths(spec: PoolSpec, seq_index: int) -> list[int]:
    """Sample lengths of one packed sequence; they sum to spec.seq_len exactly."""
    L = spec.seq_len
    rng = np.random.default_rng([spec.seed, spec.config_index, seq_index])
    big = 0
    if spec.big == "pareto":
        big = int(min(L, round(4096.0 * (1.0 + rng.pareto(1.1)))))
    elif spec.big == "fixed":
        big = int(min(L, spec.big_len))
    elif spec.big == "frac":
        big = int(min(L, round(spec.big_frac * L)))
    rest = _lognormal_fill(rng, L - big, L) if L - big > 0 else []
    if big > 0:
        pos = int(rng.integers(0, len(rest) + 1))
        rest.insert(pos, big)
    assert sum(rest) == L and min(rest) >= 1
    return rest


def pool_lengths(spec: PoolSpec) -> list[int]:
    out: list[int] = []
    for s in range(spec.n_seqs):
        out.extend(sequence_lengths(spec, s))
    return out


def cu_seqlens(lengths) -> np.ndarray:
    """int32 prefix offsets [n+1] of the samples on the pool's token axis."""
    cu = np.zeros(len(lengths) + 1, dtype=np.int64)
    np.cumsum(np.asarray(lengths, dtype=np.int64), out=cu[1:])
    assert cu[-1] < 2**31
    return cu.astype(np.int32)


# ---- the benchmark's configurations -------------------------------------------------

def config(index: int, skew: float = 0.0, seed: int = 0) -> PoolSpec:
    """The five pool shapes of the benchmark (index 1..5; `skew` selects s for index 5) and, as index 6, a pool in the
    micro-benchmark head shape of the paper's Table 1 (Hq 128 / Hkv 4 / d 256): two packed 32768-token sequences,
    the share of one worker of a 256K sequence at CP = 8."""
    if index == 1:
        return PoolSpec("tiny", 1, 1, 4096, 4, 4, 64, seed=seed)
    if index == 2:
        return PoolSpec("qwen3-8b", 2, 4, 32768, 32, 8, 128, seed=seed)
    if index == 3:
        return PoolSpec("qwen3-30b-a3b", 3, 8, 32768, 32, 4, 128, big="pareto", seed=seed)
    if index == 4:
        return PoolSpec("qwen3-235b-a22b-1m", 4, 1, 1048576, 64, 4, 128, big="fixed",
                        big_len=262144, seed=seed)
    if index == 5:
        return PoolSpec(f"skew-{skew:g}", 5, 8, 65536, 32, 8, 128,
                        big="frac" if skew > 0 else "none", big_frac=skew, seed=seed)
    if index == 6:
        return PoolSpec("microbenchmark-heads", 6, 2, 32768, 128, 4, 256, seed=seed)
    raise ValueError(f"no config {index}")


def random_layout(rng: np.random.Generator, total: int, max_len: int) -> list[int]:
    """Small random sample layout for tests: lengths in [1, max_len] summing to `total`."""
    out: list[int] = []
    left = total
    while left > 0:
        x = int(min(left, rng.integers(1, max_len + 1)))
        out.append(x)
        left -= x
    return out


# ---- tensors -------------------------------------------------------------------------

def _torch():
    import torch
    return torch


def make_tensors(total_tokens: int, hq: int, hkv: int, head_dim: int, seed: int = 0,
                 device: str = "cpu", names=("q", "k", "v", "dout"), scale: float = 1.0):
    """bf16 N(0,1) tensors in the packed "thd" layout: q, dout [T, Hq, d]; k, v [T, Hkv, d].

    Each tensor has its own generator seeded from (seed, tensor index) so that any
    subset can be regenerated alone.  On "cuda" the device generator is used, so CPU
    and GPU draws differ; parity tests copy one side's tensors to the other.
    """
    torch = _torch()
    shapes = {"q": (total_tokens, hq, head_dim), "k": (total_tokens, hkv, head_dim),
              "v": (total_tokens, hkv, head_dim), "dout": (total_tokens, hq, head_dim)}
    order = {"q": 0, "k": 1, "v": 2, "dout": 3}
    out = {}
    for nm in names:
        g = torch.Generator(device=device)
        g.manual_seed(1_000_003 * (seed + 1) + order[nm])
        t = torch.randn(shapes[nm], generator=g, device=device, dtype=torch.bfloat16)
        if scale != 1.0 and nm == "q":
            t = (t.float() * scale).to(torch.bfloat16)
        out[nm] = t
    return out
