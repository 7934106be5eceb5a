"""Multi-GPU form of the path: independent pools per rank, no data-path collective.

SH-Tiles never exchange data on one GPU, and a pool is one GPU's unit of work, so N GPUs run N
pools side by side (weak scaling).  The only cross-rank step is bookkeeping for a measurement:
the slowest rank's time and the summed work.  Backend-agnostic (NCCL on GPUs, gloo in tests).
"""
from __future__ import annotations

import dataclasses

from . import pools


def rank_spec(config_index: int, skew: float, rank: int, n_seqs: int = 0) -> pools.PoolSpec:
    """The pool a rank runs: the benchmark shape with the rank as generator seed."""
    spec = pools.config(config_index, skew, seed=rank)
    if n_seqs:
        spec = dataclasses.replace(spec, n_seqs=n_seqs, name=f"{spec.name}[{n_seqs} seqs]")
    return spec


def aggregate(ms_local: float, work_local: float, device="cpu"):
    """(max over ranks of ms_local, sum over ranks of work_local); identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(work_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    w = torch.tensor([work_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return float(t.item()), float(w.item())
