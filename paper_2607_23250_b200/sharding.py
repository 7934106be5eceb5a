"""Multi-GPU form of the path: ONE pool split over the ranks by attention heads.

Heads never exchange data inside attention, so the natural cut of a pool is along the head axis (the
paper's SH-Tiles are sequence-block x head-shard tiles, and shards of the same block "have equal work but no
KV affinity", Section 4.3.1).  Rank r of N takes the kv heads {r, r + N, ...} together with the query heads
that read them, so a GQA group is never torn apart and no rank needs another rank's tensors: no data-path
collective at all.  When there are more ranks than kv heads, the ranks that share a kv head split its
query heads between them; dK and dV of that kv head are then partial sums and are added up across those
ranks (one all-reduce in the sub-group, the only exchange step of this form).

Every rank plans and runs the whole token axis for its heads with the single-GPU library; this module only
does the bookkeeping (which heads, which sub-group, the max-time / summed-work reduction of a measurement).
Backend-agnostic: NCCL on GPUs, gloo in the CPU tests.
"""
from __future__ import annotations

import dataclasses

from . import pools


@dataclasses.dataclass(frozen=True)
class HeadShard:
    """The heads of one rank.  `q_heads` are sorted and grouped by kv head in the order of `kv_heads`,
    so slicing q[:, q_heads] and k[:, kv_heads] gives contiguous-group tensors the library accepts as they are."""
    rank: int
    world: int
    kv_heads: tuple          # global kv head indices of this rank
    q_heads: tuple           # global query head indices of this rank
    kv_sharers: tuple        # ranks that hold the same kv heads (length 1: nothing to reduce)

    @property
    def hq(self) -> int:
        return len(self.q_heads)

    @property
    def hkv(self) -> int:
        return len(self.kv_heads)


def head_groups(hq: int, hkv: int, world: int, rank: int) -> HeadShard:
    """Heads of `rank` out of `world` ranks for a layer with hq query and hkv kv heads (hkv divides hq).

    world <= hkv (world divides hkv): kv heads {rank, rank + world, ...} with all their query heads.
    world  > hkv (hkv divides world, world divides hq): kv head rank % hkv, and the (rank // hkv)-th slice of its
    query heads; the world // hkv ranks of a kv head form the sub-group that sums dK / dV."""
    if hq <= 0 or hkv <= 0 or hq % hkv or world <= 0 or not (0 <= rank < world):
        raise ValueError("bad head counts or rank")
    G = hq // hkv
    if world <= hkv:
        if hkv % world:
            raise ValueError(f"{world} ranks do not divide {hkv} kv heads")
        kv = tuple(range(rank, hkv, world))
        q = tuple(h * G + g for h in kv for g in range(G))
        return HeadShard(rank, world, kv, q, (rank,))
    if world % hkv or hq % world:
        raise ValueError(f"{world} ranks fit neither {hkv} kv heads nor {hq} query heads")
    per = world // hkv                      # ranks per kv head
    kvh, part = rank % hkv, rank // hkv
    width = G // per                        # query heads per rank
    q = tuple(kvh * G + part * width + g for g in range(width))
    return HeadShard(rank, world, (kvh,), q, tuple(kvh + hkv * s for s in range(per)))


def slice_heads(shard: HeadShard, q, k, v, dout=None):
    """The rank's contiguous [T, heads, d] slices of the full tensors (torch tensors, any device)."""
    import torch
    qi = torch.as_tensor(shard.q_heads, device=q.device)
    ki = torch.as_tensor(shard.kv_heads, device=k.device)
    out = [q.index_select(1, qi).contiguous(), k.index_select(1, ki).contiguous(), v.index_select(1, ki).contiguous()]
    if dout is not None:
        out.append(dout.index_select(1, qi).contiguous())
    return out


def reduce_kv_grads(shard: HeadShard, dk, dv, group=None):
    """Adds dK and dV up over the ranks that share this rank's kv head (no-op when there is one sharer).
    `group` is the process sub-group of shard.kv_sharers (see kv_subgroups)."""
    if len(shard.kv_sharers) == 1:
        return dk, dv
    import torch
    import torch.distributed as dist
    acc_k, acc_v = dk.float(), dv.float()          # partial sums are added in fp32, rounded once
    dist.all_reduce(acc_k, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(acc_v, op=dist.ReduceOp.SUM, group=group)
    return acc_k.to(dk.dtype), acc_v.to(dv.dtype)


def kv_subgroups(hq: int, hkv: int, world: int):
    """Creates (on every rank, in the same order, as torch.distributed requires) the sub-groups of ranks that
    share a kv head; returns {kv head: group}.  Empty when no kv head is shared."""
    if world <= hkv:
        return {}
    import torch.distributed as dist
    per = world // hkv
    return {kvh: dist.new_group([kvh + hkv * s for s in range(per)]) for kvh in range(hkv)}


def rank_spec(config_index: int, skew: float, rank: int, n_seqs: int = 0, replicas: bool = False) -> pools.PoolSpec:
    """The pool a rank works on: the same pool on every rank (head-sharded), or, with `replicas`, an
    independent pool of the same shape per rank (the rank is the generator seed)."""
    spec = pools.config(config_index, skew, seed=rank if replicas else 0)
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
