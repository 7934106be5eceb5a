"""CPU oracle of the tile exchange schedule (TEST INFRASTRUCTURE ONLY; plain loops, small pools).

Section 4.3.3 (tile exchange planning) turns an assignment sigma into tensor transfers; Section 4.4 (the
Pipeliner) moves every transfer in M equal head pieces, chunk m carrying the m-th piece of every record.
Everything here is written from those two sections and the layout readings of the pool planner: sequence s
belongs to workers s*CP .. s*CP+CP-1, worker c of the group holds the c-th run of ceil(L_s / CP) tokens; the
Q-home of a block is the worker holding its first token.

A record is (kind, src, dst, tok0, ntok, shard):
  kind 0: the Q rows [tok0, tok0 + ntok) of a tile placed away from its Q-home.  Forward: Q goes src -> dst and
          the output comes back dst -> src.  Backward: dO goes src -> dst, dQ comes back dst -> src.
  kind 1: the K and V rows [tok0, tok0 + ntok) of a KV group (sample, shard) selected for destination dst and
          held by src (one record per token run of the sample that lives on another worker; runs already at dst
          do not move; a group fetched for one destination is fetched once however many tiles there use it).
          Forward: K, V go src -> dst.  Backward: dK, dV partial sums go dst -> src and are added there.
Order: kind 0 records by tile id, then kind 1 records by (dst, sample, shard, src).
"""
from __future__ import annotations

import numpy as np


def _owner(seq_off, s, cp, tok):
    L = int(seq_off[s + 1]) - int(seq_off[s])
    run = (L + cp - 1) // cp
    return s * cp + (tok - int(seq_off[s])) // max(run, 1)


def _seq_of(seq_off, tok):
    s = 0
    while s + 1 < len(seq_off) - 1 and seq_off[s + 1] <= tok:
        s += 1
    return s


def tiles(cu, seq_off, cp, block, n_shards):
    """(q0, q1, shard, q_home, [samples with a token in the block]) of every tile, in tile-id order."""
    out = []
    n = len(cu) - 1
    for s in range(len(seq_off) - 1):
        q0 = int(seq_off[s])
        while q0 < int(seq_off[s + 1]):
            q1 = min(q0 + block, int(seq_off[s + 1]))
            js = [j for j in range(n) if max(q0, int(cu[j])) < min(q1, int(cu[j + 1]))]
            for h in range(n_shards):
                out.append((q0, q1, h, _owner(seq_off, s, cp, q0), js))
            q0 = q1
    return out


def schedule(cu, seq_off, cp, block, n_shards, sigma):
    """The transfer records implied by assignment sigma (int array over tiles) -> int32 array [n_records, 6]."""
    cu = [int(x) for x in cu]
    seq_off = [int(x) for x in seq_off]
    n = len(cu) - 1
    W = (len(seq_off) - 1) * cp
    tl = tiles(cu, seq_off, cp, block, n_shards)
    assert len(tl) == len(sigma)
    rec = []
    for t, (q0, q1, h, home, _) in enumerate(tl):
        if int(sigma[t]) != home:
            rec.append((0, home, int(sigma[t]), q0, q1 - q0, h))
    selected = [set() for _ in range(W)]                  # KV groups some tile placed at r refers to
    for t, (_, _, h, _, js) in enumerate(tl):
        for j in js:
            selected[int(sigma[t])].add((j, h))
    for r in range(W):
        for (j, h) in sorted(selected[r]):
            a, e = cu[j], cu[j + 1]
            if e <= a:
                continue
            s = _seq_of(seq_off, a)
            runs = {}                                      # owner -> [first token, one past the last] of sample j there
            for tok in range(a, e):
                w = _owner(seq_off, s, cp, tok)
                lo, hi = runs.get(w, (tok, tok))
                runs[w] = (min(lo, tok), tok + 1)
            for w in sorted(runs):
                if w != r:
                    rec.append((1, w, r, runs[w][0], runs[w][1] - runs[w][0], h))
    return np.asarray(rec, dtype=np.int32).reshape(-1, 6)


def chunk_heads(shard, m, hq, hkv, n_shards, n_chunks):
    """Heads chunk m of a record on head shard `shard` carries: (query heads, kv heads first needed by this chunk).

    The shard's hq / n_shards query heads are cut into n_chunks equal pieces (n_chunks divides that width); a kv
    head travels with the first chunk whose query heads read it (query head q reads kv head q // (hq / hkv))."""
    width = hq // n_shards
    assert width % n_chunks == 0
    piece = width // n_chunks
    G = hq // hkv
    qh = list(range(shard * width + m * piece, shard * width + (m + 1) * piece))
    seen = set()
    for mm in range(m):
        seen |= {q // G for q in range(shard * width + mm * piece, shard * width + (mm + 1) * piece)}
    kvh = sorted({q // G for q in qh} - seen)
    return qh, kvh


def chunk_bytes(records, m, hq, hkv, head_dim, n_shards, n_chunks, n_workers):
    """Forward and backward send-byte matrices [src, dst] of chunk m (bf16 tensors)."""
    fwd = np.zeros((n_workers, n_workers), np.int64)
    bwd = np.zeros((n_workers, n_workers), np.int64)
    for kind, src, dst, _, ntok, shard in records:
        qh, kvh = chunk_heads(int(shard), m, hq, hkv, n_shards, n_chunks)
        if kind == 0:
            b = int(ntok) * len(qh) * head_dim * 2
            fwd[src, dst] += b      # Q out
            fwd[dst, src] += b      # output back
            bwd[src, dst] += b      # dO along the Q path
            bwd[dst, src] += b      # dQ along the output path
        else:
            b = 2 * int(ntok) * len(kvh) * head_dim * 2
            fwd[src, dst] += b      # K and V
            bwd[dst, src] += b      # dK and dV back to where K and V came from
    return fwd, bwd
