"""Executing a tile exchange schedule across the workers of a pool (host logic above the library).

Section 4.3.3 of the paper turns the assignment into transfers, Section 4.4 (the Pipeliner) moves them in M
equal head pieces so that chunk m's compute overlaps chunk m+1's dispatch and chunk m-1's return.  This
module is that runtime's bookkeeping and message flow on torch.distributed point-to-point calls: which bytes
each pair of workers exchanges in which chunk, in what order the non-blocking sends and receives are posted,
how a worker assembles the inputs of its tiles from local rows and received rows, and how the results and
the gradients travel back.  The attention arithmetic itself is passed in as two callables, so the same flow
runs on CPU ranks in the tests and would run on GPUs with calls into the attention kernels on tensors that
have first been copied into the worker's own memory (a worker never computes on a peer's memory).

Layout (the pool planner's reading): sequence s belongs to workers s*CP .. s*CP+CP-1; worker c of the group
holds the c-th run of ceil(L_s / CP) tokens; the Q-home of a block is the worker holding its first token, and
the run length is required to be a multiple of the block size here, so a block's rows all live at its Q-home.
"""
from __future__ import annotations

import dataclasses

import numpy as np


@dataclasses.dataclass(frozen=True)
class PoolLayout:
    cu: tuple            # sample offsets of the pool's token axis, n + 1 entries
    seq_off: tuple       # packed-sequence offsets, P + 1 entries
    cp: int
    block: int
    n_shards: int
    hq: int
    hkv: int
    head_dim: int

    @property
    def n_workers(self):
        return (len(self.seq_off) - 1) * self.cp

    def run(self, w):
        """Token range [t0, t1) worker w holds."""
        s, c = divmod(w, self.cp)
        L = self.seq_off[s + 1] - self.seq_off[s]
        run = (L + self.cp - 1) // self.cp
        t0 = self.seq_off[s] + c * run
        return min(t0, self.seq_off[s + 1]), min(t0 + run, self.seq_off[s + 1])

    def owner(self, tok):
        for s in range(len(self.seq_off) - 1):
            if self.seq_off[s] <= tok < self.seq_off[s + 1]:
                L = self.seq_off[s + 1] - self.seq_off[s]
                return s * self.cp + (tok - self.seq_off[s]) // ((L + self.cp - 1) // self.cp)
        raise ValueError("token outside the pool")

    def check_aligned(self):
        for s in range(len(self.seq_off) - 1):
            L = self.seq_off[s + 1] - self.seq_off[s]
            if ((L + self.cp - 1) // self.cp) % self.block:
                raise ValueError("run length must be a multiple of the block size")

    def tiles(self):
        """[(q0, q1, shard, q_home)] in tile-id order (blocks sequence by sequence, id = block * H + shard)."""
        out = []
        for s in range(len(self.seq_off) - 1):
            q0 = self.seq_off[s]
            while q0 < self.seq_off[s + 1]:
                q1 = min(q0 + self.block, self.seq_off[s + 1])
                for h in range(self.n_shards):
                    out.append((q0, q1, h, self.owner(q0)))
                q0 = q1
        return out

    def fragments(self, q0, q1):
        """Sample fragments of the rows [q0, q1): [(sample start, sample end, first row, one past the last row)]."""
        out = []
        for j in range(len(self.cu) - 1):
            lo, hi = max(q0, self.cu[j]), min(q1, self.cu[j + 1])
            if lo < hi:
                out.append((self.cu[j], self.cu[j + 1], lo, hi))
        return out

    def chunk_heads(self, shard, m, n_chunks):
        """(query heads, kv heads first read by this chunk, kv heads read by this chunk) of chunk m on `shard`."""
        width = self.hq // self.n_shards
        if width % n_chunks:
            raise ValueError("the number of chunks must divide the shard's head width")
        piece, G = width // n_chunks, self.hq // self.hkv
        base = shard * width
        qh = list(range(base + m * piece, base + (m + 1) * piece))
        before = {q // G for q in range(base, base + m * piece)}
        reads = sorted({q // G for q in qh})
        return qh, [h for h in reads if h not in before], reads


class Worker:
    """One worker's side of the exchange: forward then backward over M head chunks.

    local: dict of this worker's rows (its token run) of q, k, v, dout: tensors [rows, heads, d].
    attn_fwd(q_rows, k, v, a)            -> (o_rows, lse_rows [heads, rows]): rows at sample positions a.. of a sample
                                            whose K/V (positions 0 .. a + rows) are given.
    attn_bwd(q_rows, k, v, o, lse, do, a) -> (dq_rows, dk, dv) for the same fragment.
    """

    def __init__(self, rank, layout: PoolLayout, sigma, records, n_chunks, local, attn_fwd, attn_bwd, dist, torch):
        layout.check_aligned()
        self.r, self.L, self.M = rank, layout, n_chunks
        self.sigma = [int(x) for x in sigma]
        self.rec = [tuple(int(x) for x in row) for row in np.asarray(records).reshape(-1, 6)]
        self.local, self.fwd_fn, self.bwd_fn, self.dist, self.torch = local, attn_fwd, attn_bwd, dist, torch
        self.t0, self.t1 = layout.run(rank)
        self.tiles = layout.tiles()
        self.mine = [t for t in range(len(self.tiles)) if self.sigma[t] == rank]
        self.store = {}        # (name, tok0, head) -> rows received from another worker, kept for the backward pass
        self.saved = {}        # (tile, chunk) -> what the backward pass needs from the forward pass

    # ---- rows: local or received ------------------------------------------------------------------
    def _rows(self, name, lo, hi, heads):
        """Rows [lo, hi) of tensor `name` for the given heads, from the local run and / or received records."""
        torch = self.torch
        parts, pos = [], lo
        while pos < hi:
            if self.t0 <= pos < self.t1:
                end = min(hi, self.t1)
                parts.append(self.local[name][pos - self.t0:end - self.t0][:, heads])
            else:
                key = next(k for k in self.store if k[0] == name and k[1] <= pos < k[1] + self.store[k].shape[0]
                           and k[2] == tuple(heads))
                buf = self.store[key]
                end = min(hi, key[1] + buf.shape[0])
                parts.append(buf[pos - key[1]:end - key[1]])
            pos = end
        return parts[0] if len(parts) == 1 else torch.cat(parts, 0)

    # ---- messages ----------------------------------------------------------------------------------
    def _peers(self, kind_filter, as_src):
        return sorted({(rc[2] if as_src else rc[1]) for rc in self.rec if kind_filter(rc) and (rc[1] if as_src else rc[2]) == self.r})

    def _post(self, stage, m, outgoing, incoming_shapes):
        """Non-blocking sends of `outgoing` {peer: [tensors]} and receives into fresh buffers of
        `incoming_shapes` {peer: [shapes]}; returns (handles, {peer: [buffers]})."""
        torch, dist = self.torch, self.dist
        handles, bufs = [], {}
        tag = stage * 64 + m
        for peer, shapes in sorted(incoming_shapes.items()):
            n = sum(int(np.prod(s)) for s in shapes)
            flat = torch.empty(n, dtype=self.local["q"].dtype)
            handles.append(dist.irecv(flat, src=peer, tag=tag))
            bufs[peer] = (flat, shapes)
        for peer, tensors in sorted(outgoing.items()):
            flat = torch.cat([t.reshape(-1) for t in tensors]) if tensors else torch.empty(0, dtype=self.local["q"].dtype)
            handles.append(dist.isend(flat.contiguous(), dst=peer, tag=tag))
        return handles, bufs

    @staticmethod
    def _unpack(bufs):
        out = {}
        for peer, (flat, shapes) in bufs.items():
            pos, lst = 0, []
            for s in shapes:
                n = int(np.prod(s))
                lst.append(flat[pos:pos + n].reshape(s))
                pos += n
            out[peer] = lst
        return out

    # ---- forward -----------------------------------------------------------------------------------
    def _dispatch_lists(self, m, names_q, names_kv):
        """What chunk m's dispatch sends and receives: kind 0 records carry `names_q` rows, kind 1 records `names_kv`
        rows of the kv heads this chunk is the first to read."""
        L, d = self.L, self.L.head_dim
        out, inc, inc_keys = {}, {}, {}
        for kind, src, dst, tok0, ntok, shard in self.rec:
            qh, kv_new, _ = L.chunk_heads(shard, m, self.M)
            items = [(nm, qh) for nm in names_q] if kind == 0 else ([(nm, kv_new) for nm in names_kv] if kv_new else [])
            for nm, heads in items:
                if src == self.r:
                    out.setdefault(dst, []).append(self.local[nm][tok0 - self.t0:tok0 - self.t0 + ntok][:, heads])
                if dst == self.r:
                    inc.setdefault(src, []).append((ntok, len(heads), d))
                    inc_keys.setdefault(src, []).append((nm, tok0, tuple(heads)))
        return out, inc, inc_keys

    def forward(self):
        """Returns this worker's rows of the output, [rows, hq, d], and of lse, [hq, rows]."""
        torch, L = self.torch, self.L
        n_rows = self.t1 - self.t0
        out = torch.zeros((n_rows, L.hq, L.head_dim), dtype=self.local["q"].dtype)
        lse = torch.zeros((L.hq, n_rows), dtype=torch.float32)
        pending_in = {}
        returns = []

        def post_dispatch(m):
            o, i, keys = self._dispatch_lists(m, ("q",), ("k", "v"))
            h, bufs = self._post(0, m, o, i)
            pending_in[m] = (h, bufs, keys)

        post_dispatch(0)
        for m in range(self.M):
            if m + 1 < self.M:
                post_dispatch(m + 1)                        # chunk m+1's inputs travel while chunk m computes
            h, bufs, keys = pending_in.pop(m)
            for x in h:
                x.wait()
            for peer, lst in self._unpack(bufs).items():
                for key, buf in zip(keys[peer], lst):
                    self.store[key] = buf
            # compute chunk m of every tile placed here
            back, back_shapes = {}, {}
            for t in self.mine:
                q0, q1, shard, home = self.tiles[t]
                qh, _, kvr = L.chunk_heads(shard, m, self.M)
                o_rows = torch.zeros((q1 - q0, len(qh), L.head_dim), dtype=self.local["q"].dtype)
                l_rows = torch.zeros((len(qh), q1 - q0), dtype=torch.float32)
                for (s0, s1, lo, hi) in L.fragments(q0, q1):
                    qf = self._rows("q", lo, hi, qh)
                    kf, vf = self._kv(s0, hi, kvr)
                    o_f, l_f = self.fwd_fn(qf, kf, vf, lo - s0)
                    o_rows[lo - q0:hi - q0] = o_f
                    l_rows[:, lo - q0:hi - q0] = l_f
                self.saved[(t, m)] = (o_rows, l_rows)
                if home == self.r:
                    out[q0 - self.t0:q1 - self.t0][:, qh] = o_rows
                    lse[qh, q0 - self.t0:q1 - self.t0] = l_rows
                else:
                    back.setdefault(home, []).extend([o_rows, l_rows])
            # chunk m's outputs go home while chunk m+1 computes; lse travels as fp32 in a second message
            returns.append(self._return_outputs(m, back))
        for handles, finish in returns:
            for x in handles:
                x.wait()
            finish(out, lse)
        return out, lse

    def _kv(self, s0, hi, kv_heads):
        k = self._rows("k", s0, hi, kv_heads)
        v = self._rows("v", s0, hi, kv_heads)
        return k, v

    def _return_outputs(self, m, back):
        """Sends chunk m's output rows of migrated tiles to their Q-homes; receives the ones computed elsewhere."""
        torch, dist, L = self.torch, self.dist, self.L
        handles = []
        tag_o, tag_l = 1 * 64 + m, 2 * 64 + m
        for peer in sorted(back):
            o_list = back[peer][0::2]
            l_list = back[peer][1::2]
            handles.append(dist.isend(torch.cat([x.reshape(-1) for x in o_list]).contiguous(), dst=peer, tag=tag_o))
            handles.append(dist.isend(torch.cat([x.reshape(-1) for x in l_list]).contiguous(), dst=peer, tag=tag_l))
        expect = {}
        for t, (q0, q1, shard, home) in enumerate(self.tiles):
            if home == self.r and self.sigma[t] != self.r:
                expect.setdefault(self.sigma[t], []).append((t, q0, q1, shard))
        bufs = {}
        for peer in sorted(expect):
            n_o = sum((q1 - q0) * len(L.chunk_heads(sh, m, self.M)[0]) * L.head_dim for _, q0, q1, sh in expect[peer])
            n_l = sum((q1 - q0) * len(L.chunk_heads(sh, m, self.M)[0]) for _, q0, q1, sh in expect[peer])
            fo = torch.empty(n_o, dtype=self.local["q"].dtype)
            fl = torch.empty(n_l, dtype=torch.float32)
            handles.append(dist.irecv(fo, src=peer, tag=tag_o))
            handles.append(dist.irecv(fl, src=peer, tag=tag_l))
            bufs[peer] = (fo, fl)

        def finish(out, lse):
            for peer, (fo, fl) in bufs.items():
                po = pl = 0
                for _, q0, q1, sh in expect[peer]:
                    qh = L.chunk_heads(sh, m, self.M)[0]
                    n = (q1 - q0) * len(qh)
                    out[q0 - self.t0:q1 - self.t0][:, qh] = fo[po:po + n * L.head_dim].reshape(q1 - q0, len(qh), L.head_dim)
                    lse[qh, q0 - self.t0:q1 - self.t0] = fl[pl:pl + n].reshape(len(qh), q1 - q0)
                    po += n * L.head_dim
                    pl += n
        return handles, finish

    # ---- backward: the same records, reversed -----------------------------------------------------------
    def backward(self):
        """Returns this worker's rows of dq [rows, hq, d], dk and dv [rows, hkv, d] (fp32 sums, then rounded once)."""
        torch, dist, L = self.torch, self.dist, self.L
        n_rows = self.t1 - self.t0
        dt = self.local["q"].dtype
        dq = torch.zeros((n_rows, L.hq, L.head_dim), dtype=dt)
        dk = torch.zeros((n_rows, L.hkv, L.head_dim), dtype=torch.float32)
        dv = torch.zeros_like(dk)
        pending_in, returns = {}, []

        def post_dispatch(m):                               # dO follows the forward Q-dispatch path
            o, i, keys = self._dispatch_lists(m, ("dout",), ())
            h, bufs = self._post(3, m, o, i)
            pending_in[m] = (h, bufs, keys)

        post_dispatch(0)
        for m in range(self.M):
            if m + 1 < self.M:
                post_dispatch(m + 1)
            h, bufs, keys = pending_in.pop(m)
            for x in h:
                x.wait()
            for peer, lst in self._unpack(bufs).items():
                for key, buf in zip(keys[peer], lst):
                    self.store[key] = buf
            dq_back = {}
            kv_acc = {}                 # (sample start, kv head, shard) -> [dk, dv] sums over the rows of the sample
            for t in self.mine:
                q0, q1, shard, home = self.tiles[t]
                qh, _, kvr = L.chunk_heads(shard, m, self.M)
                o_rows, l_rows = self.saved[(t, m)]
                dq_rows = torch.zeros((q1 - q0, len(qh), L.head_dim), dtype=dt)
                for (s0, s1, lo, hi) in L.fragments(q0, q1):
                    qf = self._rows("q", lo, hi, qh)
                    dof = self._rows("dout", lo, hi, qh)
                    kf, vf = self._kv(s0, hi, kvr)
                    dq_f, dk_f, dv_f = self.bwd_fn(qf, kf, vf, o_rows[lo - q0:hi - q0], l_rows[:, lo - q0:hi - q0], dof, lo - s0)
                    dq_rows[lo - q0:hi - q0] = dq_f
                    for x, kvh in enumerate(kvr):
                        acc = kv_acc.setdefault((s0, kvh, shard), [torch.zeros((s1 - s0, L.head_dim), dtype=torch.float32),
                                                                   torch.zeros((s1 - s0, L.head_dim), dtype=torch.float32)])
                        acc[0][:hi - s0] += dk_f[:, x].float()
                        acc[1][:hi - s0] += dv_f[:, x].float()
                if home == self.r:
                    dq[q0 - self.t0:q1 - self.t0][:, qh] = dq_rows
                else:
                    dq_back.setdefault(home, []).append(dq_rows)
            returns.append(self._return_grads(m, dq_back, kv_acc, dk, dv))
        for handles, finish in returns:
            for x in handles:
                x.wait()
            finish(dq, dk, dv)
        return dq, dk.to(dt), dv.to(dt)

    def _return_grads(self, m, dq_back, kv_acc, dk, dv):
        """dQ returns along the forward output path; dK / dV partial sums retrace the KV fetch paths and are added at
        the worker that holds the rows (partial sums travel in fp32).  Rows of this worker's own run are added here."""
        torch, dist, L = self.torch, self.dist, self.L
        handles = []
        tag_q, tag_kv = 4 * 64 + m, 5 * 64 + m
        for peer in sorted(dq_back):
            handles.append(dist.isend(torch.cat([x.reshape(-1) for x in dq_back[peer]]).contiguous(), dst=peer, tag=tag_q))
        # local part of the kv sums, and the runs that go back to other workers.  A kv head's sums leave with the LAST
        # chunk that reads it, when every query head of the shard that reads it has contributed.
        self._kv_pending = getattr(self, "_kv_pending", {})
        for key, acc in kv_acc.items():
            cur = self._kv_pending.setdefault(key, [torch.zeros_like(acc[0]), torch.zeros_like(acc[1])])
            cur[0] += acc[0]
            cur[1] += acc[1]
        out_kv = {}
        if m == self.M - 1:
            for (s0, kvh, _), (a_k, a_v) in sorted(self._kv_pending.items()):
                n = a_k.shape[0]
                lo, hi = max(s0, self.t0), min(s0 + n, self.t1)
                if lo < hi:
                    dk[lo - self.t0:hi - self.t0, kvh] += a_k[lo - s0:hi - s0]
                    dv[lo - self.t0:hi - self.t0, kvh] += a_v[lo - s0:hi - s0]
            for kind, src, dst, tok0, ntok, shard in self.rec:
                if kind == 1 and dst == self.r:
                    heads = sorted({h for mm in range(self.M) for h in L.chunk_heads(shard, mm, self.M)[1]})
                    for kvh in heads:
                        s0 = max(c for c in L.cu if c <= tok0)
                        a_k, a_v = self._kv_pending.get((s0, kvh, shard), (None, None))
                        z = torch.zeros((ntok, L.head_dim), dtype=torch.float32)
                        out_kv.setdefault(src, []).extend([a_k[tok0 - s0:tok0 - s0 + ntok] if a_k is not None else z,
                                                           a_v[tok0 - s0:tok0 - s0 + ntok] if a_v is not None else z])
            for peer in sorted(out_kv):
                handles.append(dist.isend(torch.cat([x.reshape(-1) for x in out_kv[peer]]).contiguous(), dst=peer, tag=tag_kv))
        expect_q, bufs_q = {}, {}
        for t, (q0, q1, shard, home) in enumerate(self.tiles):
            if home == self.r and self.sigma[t] != self.r:
                expect_q.setdefault(self.sigma[t], []).append((q0, q1, shard))
        for peer in sorted(expect_q):
            n = sum((q1 - q0) * len(L.chunk_heads(sh, m, self.M)[0]) * L.head_dim for q0, q1, sh in expect_q[peer])
            f = torch.empty(n, dtype=self.local["q"].dtype)
            handles.append(dist.irecv(f, src=peer, tag=tag_q))
            bufs_q[peer] = f
        expect_kv, bufs_kv = {}, {}
        if m == self.M - 1:
            for kind, src, dst, tok0, ntok, shard in self.rec:
                if kind == 1 and src == self.r:
                    heads = sorted({h for mm in range(self.M) for h in L.chunk_heads(shard, mm, self.M)[1]})
                    for kvh in heads:
                        expect_kv.setdefault(dst, []).append((tok0, ntok, kvh))
            for peer in sorted(expect_kv):
                n = sum(2 * ntok * L.head_dim for _, ntok, _ in expect_kv[peer])
                f = torch.empty(n, dtype=torch.float32)
                handles.append(dist.irecv(f, src=peer, tag=tag_kv))
                bufs_kv[peer] = f

        def finish(dq, dk, dv):
            for peer, f in bufs_q.items():
                pos = 0
                for q0, q1, sh in expect_q[peer]:
                    qh = L.chunk_heads(sh, m, self.M)[0]
                    n = (q1 - q0) * len(qh) * L.head_dim
                    dq[q0 - self.t0:q1 - self.t0][:, qh] = f[pos:pos + n].reshape(q1 - q0, len(qh), L.head_dim)
                    pos += n
            for peer, f in bufs_kv.items():
                pos = 0
                for tok0, ntok, kvh in expect_kv[peer]:
                    n = ntok * L.head_dim
                    dk[tok0 - self.t0:tok0 - self.t0 + ntok, kvh] += f[pos:pos + n].reshape(ntok, L.head_dim)
                    dv[tok0 - self.t0:tok0 - self.t0 + ntok, kvh] += f[pos + n:pos + 2 * n].reshape(ntok, L.head_dim)
                    pos += 2 * n
        return handles, finish


def library_attention(device="cuda"):
    """Attention callables for Worker that run the library's kernels on `device`.

    The Worker hands a fragment (rows at sample positions a .. a + rows of a sample whose K / V prefix it has
    assembled from local and received rows) in the worker's own memory; the fragment is copied to the device, the
    query side is padded with zero rows in front so that it becomes one whole sample of a one-sample pool, and the
    library plans and runs it.  Zero query rows with zero upstream gradient contribute nothing to dK / dV, so the
    padded call returns exactly the fragment's partial sums.  Planning a pool per fragment is the simple form: it
    serves to run the exchange with the real kernels; a production executor would batch a worker's fragments into
    one pool per chunk."""
    import torch
    from . import binding as lb

    def _plan(n, hq, hkv):
        cu = torch.tensor([0, n], dtype=torch.int32, device=device)
        return lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv, total_tokens=n)

    def _dev(x, n=None, a=0):
        y = x.to(device=device, dtype=torch.bfloat16)
        if n is None:
            return y.contiguous()
        full = torch.zeros((n,) + tuple(x.shape[1:]), dtype=torch.bfloat16, device=device)
        full[a:] = y
        return full

    def fwd(qf, k, v, a):
        n = k.shape[0]
        plan = _plan(n, qf.shape[1], k.shape[1])
        out, lse = lb.libra_attn_pool_fwd(_dev(qf, n, a), _dev(k), _dev(v), plan)
        torch.cuda.synchronize()
        plan.busy_times(lb.KERNEL_FWD)
        plan.destroy()
        return out[a:].to("cpu", qf.dtype), lse[:, a:].cpu()

    def bwd(qf, k, v, o, lse, do, a):
        n = k.shape[0]
        plan = _plan(n, qf.shape[1], k.shape[1])
        lse_full = torch.zeros((qf.shape[1], n), dtype=torch.float32, device=device)
        lse_full[:, a:] = lse.to(device)
        dq, dk, dv = lb.libra_attn_pool_bwd(_dev(qf, n, a), _dev(k), _dev(v), _dev(o, n, a), lse_full, _dev(do, n, a), plan)
        torch.cuda.synchronize()
        plan.busy_times(lb.KERNEL_BWD_DQ)
        plan.destroy()
        return dq[a:].to("cpu", qf.dtype), dk.to("cpu", qf.dtype), dv.to("cpu", qf.dtype)

    return fwd, bwd
