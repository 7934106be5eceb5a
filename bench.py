#!/usr/bin/env python
"""Benchmark of the pool-attention hot path (plan reused; forward + backward per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference] [--sweep]
                    [--backward fused|two-kernel]

One step = one forward + backward pass of causal, sample-masked attention over one synthetic
pool (default: the Qwen3-8B-shaped pool, 4 packed sequences x 32768 tokens, Hq 32 / Hkv 8 /
d 128).  The metric is useful TFLOP/s: 14 * d * Hq * sum_j l_j (l_j + 1) / 2 per step divided
by the step time (4 d per causal pair forward, 10 d backward).  With N > 1 (torchrun) the SAME
pool is split over the ranks by attention heads (kv heads with their query heads; strong
scaling, no data-path collective while N <= Hkv); `--replicas` runs one independent pool per
rank instead (weak scaling).  The backward runs in its fused form (one kernel over pair tiles, five GEMMs per cell)
unless `--backward two-kernel` asks for the dK/dV + dQ pair of kernels (seven GEMMs per cell, bit-reproducible).

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample
of the same workload instead.  `--sweep` prints a table over head shards x tile weights x pools.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_23250_b200 import pools, sharding  # noqa: E402

METRIC = "useful attention TFLOP/s fwd+bwd (sum of per-sample causal FLOPs)"


def kernel_ids(lb, fused, d=128):
    """name -> library kernel id of the launches of one step, and the names that keep per-CTA busy times."""
    if d == 256:   # forward pass, row statistics, dV + dK passes, dQ pass (+ rounding of dK / dV with a pair-tile plan)
        ids = {"fwd": lb.KERNEL_FWD, "bwd_prep": lb.KERNEL_BWD_PREP, "bwd_dkdv": lb.KERNEL_BWD_DKDV, "bwd_dq": lb.KERNEL_BWD_DQ}
        if fused:
            ids["bwd_post"] = lb.KERNEL_BWD_POST
        return ids, ("fwd", "bwd_dkdv", "bwd_dq")
    if fused:
        return ({"fwd": lb.KERNEL_FWD, "bwd_prep": lb.KERNEL_BWD_PREP, "bwd_fused": lb.KERNEL_BWD_FUSED,
                 "bwd_post": lb.KERNEL_BWD_POST}, ("fwd", "bwd_fused"))
    return ({"fwd": lb.KERNEL_FWD, "bwd_prep": lb.KERNEL_BWD_PREP, "bwd_dkdv": lb.KERNEL_BWD_DKDV,
             "bwd_dq": lb.KERNEL_BWD_DQ}, ("fwd", "bwd_dkdv", "bwd_dq"))


def useful_flops(lengths, hq, d):
    l = np.asarray(lengths, dtype=np.int64)
    pairs = int((l * (l + 1) // 2).sum())
    return 4 * d * hq * pairs, 10 * d * hq * pairs


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(burst=float(p["bf16_tflops"]), sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    hbm=float(p["hbm_gbs"]), source="measured")
    return dict(burst=1590.0, sustained=1400.0, hbm=6650.0, source="fallback")


# ---- clocks ------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        try:
            for line in open(self.path):
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
                except ValueError:
                    continue
                for nm, v in zip(names, parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(pw),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ---- the CPU oracle leg -------------------------------------------------------------------

def oracle_sample(spec, lengths, pair_budget=2.0e7):
    """Bounded sample of the workload for the CPU oracle: the pool's first samples, in order,
    up to `pair_budget` causal pairs, on kv head 0 and its group of query heads."""
    take, pairs = [], 0
    for l in lengths:
        p = l * (l + 1) // 2
        if pairs + p > pair_budget:                 # cut the sample that crosses the budget
            l = int((2 * (pair_budget - pairs)) ** 0.5)
            p = l * (l + 1) // 2
            if l >= 1:
                take.append(int(l)); pairs += p
            break
        take.append(int(l)); pairs += p
    G = spec.hq // spec.hkv
    desc = (f"first {len(take)} samples ({sum(take)} tokens, {pairs:.3g} causal pairs) of the pool, "
            f"kv head 0 with its {G} query heads, fwd+bwd, fp32")
    return take, G, desc


def time_oracle(spec, lengths, steps=1, warmup=0):
    import oracle
    take, G, desc = oracle_sample(spec, lengths)
    T = sum(take)
    t = pools.make_tensors(T, G, 1, spec.head_dim, seed=0)
    f = {k: v.float().numpy() for k, v in t.items()}
    cu = pools.cu_seqlens(take)
    ff, fb = useful_flops(take, G, spec.head_dim)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        o, l = oracle.attn_fwd(f["q"], f["k"], f["v"], cu)
        oracle.attn_bwd(f["q"], f["k"], f["v"], o, l, f["dout"], cu)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    cores = len(os.sched_getaffinity(0))
    return dict(value=(ff + fb) / sec / 1e12, unit="TFLOP/s", cores=cores, kind="oracle", sample=desc,
                seconds_per_step=sec)


# ---- one pool on this rank's GPU ---------------------------------------------------------------

class Pool:
    """Device tensors, plan and buffers of one pool (or of this rank's head slice of it)."""

    def __init__(self, lb, spec, dev, shard=None, weight_model="pairs", heads=0, seed=0, fused=True):
        import torch
        self.lb, self.spec, self.dev, self.shard = lb, spec, dev, shard
        self.fused = fused and spec.head_dim in (128, 256)   # a pair-tile plan: fused backward at head_dim 128,
                                                             # dV / dK passes over pair tiles at head_dim 256
        self.lengths = pools.pool_lengths(spec)
        cu_np = pools.cu_seqlens(self.lengths)
        T, d = spec.total_tokens, spec.head_dim
        t = pools.make_tensors(T, spec.hq, spec.hkv, d, seed=seed, device=str(dev))
        if shard is not None and shard.world > 1:
            q, k, v, dout = sharding.slice_heads(shard, t["q"], t["k"], t["v"], t["dout"])
            del t
        else:
            q, k, v, dout = t["q"], t["k"], t["v"], t["dout"]
        self.inp = dict(q=q, k=k, v=v, dout=dout)
        self.hq, self.hkv, self.T, self.d = q.shape[1], k.shape[1], T, d
        self.ff, self.fb = useful_flops(self.lengths, self.hq, d)
        self.cu = torch.from_numpy(cu_np).to(dev)
        self.heads = heads or self.hq
        self.blocks = weight_model == "blocks"
        self.plan = None
        self.out = dict(out=torch.empty_like(q), lse=torch.empty((self.hq, T), dtype=torch.float32, device=dev),
                        dq=torch.empty_like(q), dk=torch.empty_like(k), dv=torch.empty_like(v))

    def make_plan(self, blocks=None):
        lb = self.lb
        blocks = self.blocks if blocks is None else blocks
        directions = lb.LIBRA_DIR_Q | (lb.LIBRA_DIR_PAIR if self.fused else lb.LIBRA_DIR_KV)
        return lb.libra_plan_tiles(self.cu, self.heads, 256, directions=directions, tile_kv=128, n_heads_kv=self.hkv,
                                   total_tokens=self.T,
                                   weight_model=lb.LIBRA_WEIGHT_BLOCKS if blocks else lb.LIBRA_WEIGHT_PAIRS,
                                   unit_cost_q=12 if blocks else 0, unit_cost_kv=6 if blocks else 0)

    def build(self):
        import torch
        self.make_plan().destroy()                     # first call pays for the module load
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        self.plan = self.make_plan()                   # built once, outside the timed steps (the paper reuses it across layers)
        e1.record()
        torch.cuda.synchronize()
        assert self.plan.status() == 0
        self.ws = torch.empty(self.lb.libra_attn_pool_bwd_workspace_bytes(self.plan, self.inp["q"], self.inp["k"]),
                              dtype=torch.uint8, device=self.dev)
        return e0.elapsed_time(e1)

    def step_on(self, i, o, plan=None):
        lb, plan = self.lb, plan or self.plan
        lb.libra_attn_pool_fwd(i["q"], i["k"], i["v"], plan, out=o["out"], lse=o["lse"])
        lb.libra_attn_pool_bwd(i["q"], i["k"], i["v"], o["out"], o["lse"], i["dout"], plan, dq=o["dq"], dk=o["dk"],
                               dv=o["dv"], workspace=self.ws)

    def step(self, plan=None):
        self.step_on(self.inp, self.out, plan)

    def timed(self, steps, warmup, barrier, plan=None):
        """(ms per step, per-kernel mean ms, busy max/mean per kernel, launches) of `steps` steps between two events;
        the library records its own events around every kernel inside the same loop."""
        import torch
        lb, plan = self.lb, plan or self.plan
        for _ in range(warmup):
            self.step(plan)
        barrier()
        plan.set_timing(True)                          # fresh record: only the timed steps below
        ids, with_busy = kernel_ids(lb, self.fused, self.d)
        n0 = lb.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            self.step(plan)
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1) / steps
        self.launches = lb.launch_count() - n0
        kern = {n: statistics.mean(plan.kernel_times_ms(k)) for n, k in ids.items()}
        plan.set_timing(False)
        busy = {}
        for n in with_busy:
            which = lb.KERNEL_BWD_FUSED if (n == "bwd_dkdv" and self.fused) else ids[n]   # the lists the passes walked
            b = plan.busy_times(which).astype(np.float64)
            b = b[b > 0]
            busy[n] = round(float(b.max() / b.mean()), 4)
        return ms, kern, busy

    def tile_time_corr(self, plan=None):
        """Pearson correlation between the plan's tile weights and the time the last launch spent on each tile
        (forward: query-major tiles; fused backward: pair tiles); the paper notes that a FLOPs-balanced assignment
        need not be time-balanced."""
        lb, plan = self.lb, plan or self.plan
        out = {}
        legs = [("fwd", lb.KERNEL_FWD, lb.LIBRA_DIR_Q)]
        if self.fused and self.d == 128:
            legs.append(("bwd_fused", lb.KERNEL_BWD_FUSED, lb.LIBRA_DIR_PAIR))
        if self.d == 256:
            return out                                 # the 256-wide kernel keeps no per-tile times
        for name, kern, direction in legs:
            ns = plan.tile_times(kern).astype(np.float64)
            w = plan.export(direction)["weight"].astype(np.float64)
            ran = ns > 0
            if ran.sum() > 2 and w[ran].std() > 0 and ns[ran].std() > 0:
                out[name] = round(float(np.corrcoef(w[ran], ns[ran])[0, 1]), 4)
        return out

    def destroy(self):
        if self.plan is not None:
            self.plan.destroy()
            self.plan = None
        self.inp = self.out = self.ws = None


def pool_line(pool, ms, kern, busy):
    """Compact record of one pool's measurement (the skewed-pool and sweep legs)."""
    ff, fb = pool.ff, pool.fb
    return {"useful_tflops": round((ff + fb) / (ms * 1e-3) / 1e12, 1), "ms_per_step": round(ms, 3),
            "kernel_ms": {n: round(v, 3) for n, v in kern.items()}, "busy_max_over_mean": busy}


# ---- our arm ---------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_23250_b200 import binding as lb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    spec = sharding.rank_spec(args.config, args.skew, rank, args.seqs, replicas=args.replicas)
    shard = None if (args.replicas or world == 1) else sharding.head_groups(spec.hq, spec.hkv, world, rank)
    groups = {} if shard is None else sharding.kv_subgroups(spec.hq, spec.hkv, world)
    pool = Pool(lb, spec, dev, shard=shard, weight_model=args.weight_model, heads=args.heads,
                seed=rank if args.replicas else 0, fused=args.backward == "fused")
    plan_ms = pool.build()
    kv_shared = shard is not None and len(shard.kv_sharers) > 1

    if kv_shared:                                      # ranks sharing a kv head add their dK / dV up every step
        plain_step_on = pool.step_on
        group = groups[shard.kv_heads[0]]

        def step_on(i, o, plan=None):
            plain_step_on(i, o, plan)
            dk, dv = sharding.reduce_kv_grads(shard, o["dk"], o["dv"], group)
            o["dk"].copy_(dk); o["dv"].copy_(dv)
        pool.step_on = step_on

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K steps between events, the library's per-kernel events inside the same loop
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_local, kern, busy = pool.timed(args.steps, max(args.warmup, 3), barrier)
    launches = pool.launches
    corr = pool.tile_time_corr()
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step, work = sharding.aggregate(ms_local, float(pool.ff + pool.fb), device=dev)
    value = work / (ms_per_step * 1e-3) / 1e12

    # ---- the same steps under the plan's other tile weight (context for the busy-time spread, not the headline)
    alt = None
    if world == 1 and not args.skip_e2e:
        other = not pool.blocks
        plan2 = pool.make_plan(blocks=other)
        ms2, _, busy2 = pool.timed(args.steps, 3, barrier, plan=plan2)
        alt = {"tile_weight": "blocks (time proxy)" if other else "causal pairs (Eq. 6)",
               "value": round((pool.ff + pool.fb) / (ms2 * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
               "busy_max_over_mean": busy2, "tile_time_weight_corr": pool.tile_time_corr(plan2)}
        plan2.destroy()

    e2e = None
    if not args.skip_e2e:
        e2e = run_e2e(args, pool.step_on, barrier, pool.inp, pool.out, dev, pool.ff + pool.fb)

    line = None
    if rank == 0:
        line = headline(args, world, spec, pool, value, ms_per_step, ms_local, kern, busy, clocks, launches, e2e,
                        plan_ms, alt, shard)
        line["tile_time_weight_corr"] = corr
    pool.destroy()
    del pool
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.skip_skewed:
        line["skewed_pools"] = skewed_pools(args, lb, dev, barrier)
    if rank == 0 and world == 1 and not args.skip_cpu:
        cb = time_oracle(spec, pools.pool_lengths(spec))
        line["cpu_baseline"] = {k2: (round(v2, 6) if isinstance(v2, float) else v2) for k2, v2 in cb.items()}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def skewed_pools(args, lb, dev, barrier):
    """The pools that carry the busy-time target: the 30B-shaped pool with Pareto-tailed samples, the 1M-token
    pool with one 262144-token sample, and the skew sweep at every skew; a few steps each.  Last, the pool in the
    micro-benchmark head shape (Hq 128 / Hkv 4 / d 256), which runs the 256-wide kernels."""
    import torch
    out = {}
    for name, cfg, skew, steps in (("config3", 3, 0.0, 5), ("config5_skew0", 5, 0.0, 5), ("config5_skew0.25", 5, 0.25, 4),
                                   ("config5_skew0.5", 5, 0.5, 3), ("config5_skew1", 5, 1.0, 2), ("config4", 4, 0.0, 2),
                                   ("config6_d256", 6, 0.0, 2)):
        spec = pools.config(cfg, skew)
        pool = Pool(lb, spec, dev, weight_model=args.weight_model, fused=args.backward == "fused")
        pool.build()
        ms, kern, busy = pool.timed(steps, 1 if cfg == 4 else 2, barrier)
        rec = pool_line(pool, ms, kern, busy)
        rec["tile_time_weight_corr"] = pool.tile_time_corr()
        rec.update(steps=steps, samples=len(pool.lengths), max_sample=int(max(pool.lengths)), tokens=spec.total_tokens,
                   heads=f"Hq {spec.hq} / Hkv {spec.hkv}")
        out[name] = rec
        pool.destroy()
        del pool
        torch.cuda.empty_cache()
    return out


def run_e2e(args, step_on, barrier, dev_in, dev_out, dev, flops):
    """End to end through the public calls with HOST buffers: every step its inputs are copied from pinned host
    memory and its results are copied back.  The copies of neighbouring steps overlap the kernels of the current
    one (two device buffer sets, one copy-in and one copy-out stream), as a caller streaming batches would do."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    host_in = {n: torch.empty(x.shape, dtype=x.dtype).pin_memory().copy_(x) for n, x in dev_in.items()}
    host_out = {n: torch.empty(x.shape, dtype=x.dtype).pin_memory() for n, x in dev_out.items()}
    h2d = sum(x.numel() * x.element_size() for x in host_in.values())
    d2h = sum(x.numel() * x.element_size() for x in host_out.values())
    ins = [dev_in, {n: torch.empty_like(x) for n, x in dev_in.items()}]
    outs = [dev_out, {n: torch.empty_like(x) for n, x in dev_out.items()}]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]     # inputs of the set have landed
    ev_done = [torch.cuda.Event() for _ in range(2)]   # kernels that used the set have finished
    ev_out = [torch.cuda.Event() for _ in range(2)]    # results of the set have been copied out

    def copy_in(b):
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[b])                # the kernels that read this set before are done
            for n in ins[b]:
                ins[b][n].copy_(host_in[n], non_blocking=True)
            ev_in[b].record(s_in)

    def run(n_steps, timed):
        for ev in ev_done + ev_out:
            ev.record(main)
        torch.cuda.synchronize()
        if timed:
            e0.record(s_in)
        copy_in(0)
        for i in range(n_steps):
            b = i & 1
            if i + 1 < n_steps:
                copy_in(b ^ 1)
            main.wait_event(ev_in[b])
            main.wait_event(ev_out[b])                 # the previous results in this set have been copied out
            step_on(ins[b], outs[b])
            ev_done[b].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[b])
                for n in outs[b]:
                    host_out[n].copy_(outs[b][n], non_blocking=True)
                ev_out[b].record(s_out)
        if timed:
            s_out.wait_stream(s_in)
            e1.record(s_out)
        torch.cuda.synchronize()

    run(2, False)
    barrier()
    n_e2e = max(2, min(args.steps, 20))                 # K steps, like the device-resident leg (bounded: 65 ms each)
    run(n_e2e, True)
    barrier()
    e2e_ms, work = sharding.aggregate(e0.elapsed_time(e1) / n_e2e, float(flops), device=dev)
    return {"value": round(work / (e2e_ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 3), "steps": n_e2e}


def headline(args, world, spec, pool, value, ms_per_step, ms_local, kern, busy, clocks, launches, e2e, plan_ms, alt,
             shard):
    peaks = measured_peaks()
    hq, hkv, d, T = spec.hq, spec.hkv, spec.head_dim, spec.total_tokens
    ff, fb = pool.ff, pool.fb                      # this rank's heads
    kf = kern["fwd"]
    bwd_ms = sum(v for n, v in kern.items() if n != "fwd")
    # Dominant kernel: the backward's main kernel.  Algorithmic work per launch of the fused kernel: the five GEMMs
    # of the gradient (S, dP, dV, dK, dQ = 10 d flops per causal pair per query head, all of them useful); of the
    # dK/dV kernel of the two-kernel form: the four GEMMs it owns (8 d).  It is timed inside the timed region; that
    # region's length decides which measured peak applies (burst under a second, else sustained).
    if pool.fused and d == 128:
        dom, dom_ms, fa = "k_attn_bwd_fused", kern["bwd_fused"], fb
        executed = {"fused (10 d per pair)": round(fb / kern["bwd_fused"] / 1e9, 1)}
        ratio = "14 d / 14 d per causal pair (every GEMM of the gradient is computed once)"
    elif d == 256:
        # the 256-wide kernel: dV pass (S, dV) + dK pass (S, dP, dK) = 10 d executed, dQ pass (S, dP, dQ) = 6 d
        dom, dom_ms, fa = "k_attn_d256 (dV and dK passes)", kern["bwd_dkdv"], fb
        executed = {"dv + dk passes (10 d per pair)": round(fa / kern["bwd_dkdv"] / 1e9, 1),
                    "dq pass (6 d per pair)": round(fb * 6 // 10 / kern["bwd_dq"] / 1e9, 1)}
        ratio = "20 d / 14 d per causal pair (three gradient passes, each recomputes S)"
    else:
        dom, dom_ms, fa = "k_attn_bwd_dkdv", kern["bwd_dkdv"], fb * 8 // 10
        executed = {"dkdv (8 d per pair)": round(fa / kern["bwd_dkdv"] / 1e9, 1),
                    "dq (6 d per pair)": round(fb * 6 // 10 / kern["bwd_dq"] / 1e9, 1)}
        ratio = "18 d / 14 d per causal pair (S and dP are computed by both backward kernels)"
    ach = fa / (dom_ms * 1e-3) / 1e12
    region_s = ms_local * args.steps * 1e-3
    kind = "burst" if region_s < 1.0 else "sustained"
    peak = peaks[kind]
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4),
        "higher_is_better": True, "scaling": "weak" if (args.replicas or world == 1) else "strong",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"config {args.config}: {spec.name} pool, {spec.n_seqs} x {spec.seq_len} tokens, "
                               f"{len(pool.lengths)} samples (log-normal median 644, sigma 1.6), Hq {hq} / Hkv {hkv} / d {d}, "
                               f"causal per sample, fwd+bwd; plan built once and reused",
                   "backward": ("fused: one kernel over pair tiles (key block x %d-token query chunk x kv head), fp32 "
                                "accumulators" % pool.plan.export_pairs()[2]) if (pool.fused and d == 128) else
                               (("three passes of the 256-wide kernel (dV, dK, dQ)" + (", dV and dK over pair tiles with fp32 "
                                 "accumulators" if pool.fused else "")) if d == 256 else "two kernels (dK/dV, dQ)"),
                   "tile_q": 256, "tile_kv": 128, "head_shards": pool.heads, "n_workers": pool.plan.info()["n_workers"],
                   "tile_weight": "blocks (time proxy)" if pool.blocks else "causal pairs (Eq. 6)",
                   "l2": "inputs larger than L2 (Q alone is %.2f GB per rank)" % (pool.inp["q"].numel() * 2 / 1e9),
                   "parallelism": ("one GPU" if world == 1 else
                                   (f"{world} independent pools (seed = rank)" if args.replicas else
                                    f"one pool split by heads over {world} ranks: {shard.hkv} kv / {shard.hq} query heads per rank"
                                    + (", dK/dV summed over the ranks of a kv head" if len(shard.kv_sharers) > 1 else
                                       ", no data-path collective")))},
        "pct_of_bf16_peak": {"burst_measured": round(100 * value / world / peaks["burst"], 2),
                             "sustained_measured": round(100 * value / world / peaks["sustained"], 2),
                             "nominal_2250": round(100 * value / world / 2250.0, 2), "peaks": peaks["source"]},
        "kernel_ms_in_timed_loop": {n: round(v, 4) for n, v in kern.items()},
        "kernel_ms_sum": round(kf + bwd_ms, 4),
        "fwd_useful_tflops": round(ff / kf / 1e9, 1),
        "bwd_useful_tflops": round(fb / bwd_ms / 1e9, 1),
        "bwd_executed_tflops": executed,
        "busy_max_over_mean": busy,
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "plan_ms": round(plan_ms, 3),
        "other_tile_weight": alt,
        "roofline": {"bound": "tensor", "kernel": dom, "achieved": round(ach, 1),
                     "peak": peak, "unit": "TFLOP/s", "frac": round(ach / peak, 4),
                     "peak_kind": f"bf16 {kind}, {peaks['source']} (timed region {region_s:.2f} s)",
                     "traffic": read_traffic(dom, args),
                     "frac_of_burst": round(ach / peaks["burst"], 4),
                     "frac_of_sustained": round(ach / peaks["sustained"], 4),
                     "whole_path": {"useful_tflops_per_gpu": round(value / world, 1),
                                    "frac_of_burst": round(value / world / peaks["burst"], 4),
                                    "frac_of_sustained": round(value / world / peaks["sustained"], 4),
                                    "executed_over_useful_flops": ratio}},
    }
    return line


def read_traffic(kernel, args):
    """DRAM bytes per launch of `kernel` from the committed ncu summary (profiles/dram_traffic.txt:
    lines `kernel config seqs bytes`), scaled by nothing: only an exact workload match is used."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        for line in open(path):
            parts = line.split()
            if len(parts) >= 4 and parts[0] == kernel and int(parts[1]) == args.config and int(parts[2]) == args.seqs:
                return int(float(parts[3]))
    except Exception:
        pass
    return None


# ---- head-shard x tile-weight sweep -----------------------------------------------------------------

def run_sweep(args):
    """Useful TFLOP/s and busy-time spread against the number of head shards H and the tile weight, on the
    8B-shaped, the 30B-shaped and two skewed pools (a few steps each).  Prints a markdown table."""
    import torch
    from paper_2607_23250_b200 import binding as lb
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)

    def barrier():
        torch.cuda.synchronize()

    rows = []
    for name, cfg, skew, steps in (("config 2 (8B shape)", 2, 0.0, 8), ("config 3 (30B shape)", 3, 0.0, 4),
                                   ("config 5, skew 0.5", 5, 0.5, 2), ("config 5, skew 1", 5, 1.0, 2)):
        spec = pools.config(cfg, skew)
        for H in sorted({spec.hkv, 2 * spec.hkv, spec.hq}):
            for wm in ("pairs", "blocks"):
                for fused in (False, True):
                    pool = Pool(lb, spec, dev, weight_model=wm, heads=H, fused=fused)
                    plan_ms = pool.build()
                    ms, kern, busy = pool.timed(steps, 2, barrier)
                    rec = pool_line(pool, ms, kern, busy)
                    rows.append((name, H, wm, "fused" if fused else "two-kernel", rec, plan_ms))
                    pool.destroy()
                    del pool
                    torch.cuda.empty_cache()
    print("| pool | head shards H (forward, dQ) | tile weight | backward | useful TFLOP/s | ms/step | kernel ms | busy max/mean | plan ms |")
    print("|---|---|---|---|---|---|---|---|---|")
    for name, H, wm, form, r, plan_ms in rows:
        k = ", ".join(f"{n} {v}" for n, v in r["kernel_ms"].items())
        b = ", ".join(f"{n} {v}" for n, v in r["busy_max_over_mean"].items())
        print(f"| {name} | {H} | {wm} | {form} | {r['useful_tflops']} | {r['ms_per_step']} | {k} | {b} | {plan_ms:.1f} |")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = pools.config(args.config, args.skew, seed=0)
    lengths = pools.pool_lengths(spec)
    cb = time_oracle(spec, lengths, steps=max(1, min(args.steps, 3)), warmup=min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": round(cb["value"], 6), "unit": "TFLOP/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": max(1, min(args.steps, 3)),
        "warmup": min(args.warmup, 1), "ms_per_step": round(cb["seconds_per_step"] * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"config {args.config}: {spec.name} pool (bounded sample, CPU oracle)"},
        "cpu_baseline": {"value": round(cb["value"], 6), "unit": "TFLOP/s", "cores": cb["cores"], "kind": "oracle",
                         "sample": cb["sample"]},
        "e2e": {"value": round(cb["value"], 6), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--skew", type=float, default=0.0)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--weight-model", default="pairs", choices=["pairs", "blocks"],
                    help="tile weight of the plan: the paper's pair count, or the executed-block count")
    ap.add_argument("--backward", default="fused", choices=["fused", "two-kernel"],
                    help="backward form: one fused kernel over pair tiles (default) or the dK/dV + dQ kernels")
    ap.add_argument("--heads", type=int, default=0, help="head shards H of the query-major tiles (0 = one per query head)")
    ap.add_argument("--seqs", type=int, default=0, help="override the number of packed sequences (profiling runs)")
    ap.add_argument("--replicas", action="store_true", help="N > 1: one independent pool per rank instead of one pool split by heads")
    ap.add_argument("--sweep", action="store_true", help="print the head-shard x tile-weight table instead of the JSON line")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU oracle leg (profiling runs)")
    ap.add_argument("--skip-skewed", action="store_true", help="skip the skewed-pool leg (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
