#!/usr/bin/env python
"""Benchmark of the pool-attention hot path (plan reused; forward + backward per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

One step = one forward + backward pass of causal, sample-masked attention over one synthetic
pool (default: the Qwen3-8B-shaped pool, 4 packed sequences x 32768 tokens, Hq 32 / Hkv 8 /
d 128).  The metric is useful TFLOP/s: 14 * d * Hq * sum_j l_j (l_j + 1) / 2 per step divided
by the step time (4 d per causal pair forward, 10 d backward).  With N > 1 (torchrun) every
rank runs its own pool of the same shape (weak scaling, no data-path collective).

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample
of the same workload instead.
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


# ---- our arm ---------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_23250_b200 import binding as lb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    spec = sharding.rank_spec(args.config, args.skew, rank, args.seqs)       # every rank its own pool
    lengths = pools.pool_lengths(spec)
    cu_np = pools.cu_seqlens(lengths)
    T, hq, hkv, d = spec.total_tokens, spec.hq, spec.hkv, spec.head_dim
    ff, fb = useful_flops(lengths, hq, d)
    dev = torch.device("cuda", local)

    t = pools.make_tensors(T, hq, hkv, d, seed=rank, device=f"cuda:{local}")
    q, k, v, dout = t["q"], t["k"], t["v"], t["dout"]
    cu = torch.from_numpy(cu_np).to(dev)
    blocks = args.weight_model == "blocks"

    def make_plan():
        return lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv, total_tokens=T,
                                   weight_model=lb.LIBRA_WEIGHT_BLOCKS if blocks else lb.LIBRA_WEIGHT_PAIRS,
                                   unit_cost_q=12 if blocks else 0, unit_cost_kv=6 if blocks else 0)

    make_plan().destroy()                     # first call pays for the module load
    torch.cuda.synchronize()
    pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pe0.record()
    plan = make_plan()                        # built once, outside the timed steps (the paper reuses it across layers)
    pe1.record()
    torch.cuda.synchronize()
    plan_ms = pe0.elapsed_time(pe1)
    assert plan.status() == 0
    plan.set_timing(True)
    out = torch.empty_like(q)
    lse = torch.empty((hq, T), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(lb.libra_attn_pool_bwd_workspace_bytes(plan, q, k), dtype=torch.uint8, device=dev)

    def step_on(i, o):
        lb.libra_attn_pool_fwd(i["q"], i["k"], i["v"], plan, out=o["out"], lse=o["lse"])
        lb.libra_attn_pool_bwd(i["q"], i["k"], i["v"], o["out"], o["lse"], i["dout"], plan, dq=o["dq"], dk=o["dk"],
                               dv=o["dv"], workspace=ws)

    def step():
        step_on(dict(q=q, k=k, v=v, dout=dout), dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- device-resident timing: K steps between events, plus per-kernel events per step
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = lb.launch_count()
    kern_f, kern_b, kern_q = [], [], []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    total_ms = e0.elapsed_time(e1)
    launches = lb.launch_count() - n0
    # kernel-only durations (events recorded by the library on the launch stream), untimed extra steps
    for _ in range(min(args.steps, 5)):
        step()
        kern_f.append(plan.kernel_time_ms(lb.KERNEL_FWD))
        kern_b.append(plan.kernel_time_ms(lb.KERNEL_BWD_DKDV))
        kern_q.append(plan.kernel_time_ms(lb.KERNEL_BWD_DQ))
    clocks = sampler.stop() if rank == 0 else None
    busy_f = plan.busy_times(lb.KERNEL_FWD).astype(np.float64)
    busy_b = plan.busy_times(lb.KERNEL_BWD_DKDV).astype(np.float64)
    busy_q = plan.busy_times(lb.KERNEL_BWD_DQ).astype(np.float64)

    ms_per_step, work = sharding.aggregate(total_ms / args.steps, float(ff + fb), device=dev)
    value = work / (ms_per_step * 1e-3) / 1e12

    # ---- the same steps under the plan's other tile weight (context for the busy-time spread, not the headline)
    alt = None
    if world == 1 and not args.skip_e2e:
        other = not blocks
        plan2 = lb.libra_plan_tiles(cu, hq, 256, tile_kv=128, n_heads_kv=hkv, total_tokens=T,
                                    weight_model=lb.LIBRA_WEIGHT_BLOCKS if other else lb.LIBRA_WEIGHT_PAIRS,
                                    unit_cost_q=12 if other else 0, unit_cost_kv=6 if other else 0)

        def step2():
            lb.libra_attn_pool_fwd(q, k, v, plan2, out=out, lse=lse)
            lb.libra_attn_pool_bwd(q, k, v, out, lse, dout, plan2, dq=dq, dk=dk, dv=dv, workspace=ws)

        for _ in range(3):
            step2()
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(args.steps):
            step2()
        a1.record()
        barrier()
        spread = [plan2.busy_times(kk).astype(np.float64) for kk in (lb.KERNEL_FWD, lb.KERNEL_BWD_DKDV, lb.KERNEL_BWD_DQ)]
        alt = {"tile_weight": "blocks (time proxy)" if other else "causal pairs (Eq. 6)",
               "value": round((ff + fb) / (a0.elapsed_time(a1) / args.steps * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
               "busy_max_over_mean": {n: round(float(b.max() / b.mean()), 4) for n, b in zip(("fwd", "bwd_dkdv", "bwd_dq"), spread)}}
        plan2.destroy()

    e2e = None
    if not args.skip_e2e:
        e2e = run_e2e(args, step_on, barrier, dict(q=q, k=k, v=v, dout=dout),
                      dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv), world, dev, ff + fb)
    finish(args, rank, world, spec, lengths, plan, value, ms_per_step, (kern_f, kern_b, kern_q),
           (busy_f, busy_b, busy_q), clocks, launches, e2e, ff, fb, q, plan_ms, alt)
    plan.destroy()
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, step_on, barrier, dev_in, dev_out, world, dev, flops):
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
    n_e2e = max(2, min(args.steps, 6))
    run(n_e2e, True)
    barrier()
    e2e_ms, work = sharding.aggregate(e0.elapsed_time(e1) / n_e2e, float(flops), device=dev)
    return {"value": round(work / (e2e_ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 3)}


def finish(args, rank, world, spec, lengths, plan, value, ms_per_step, kern, busy, clocks, launches, e2e, ff, fb, q,
           plan_ms=None, alt=None):
    kern_f, kern_b, kern_q = kern
    busy_f, busy_b, busy_q = busy
    from paper_2607_23250_b200 import binding as lb  # noqa: F401
    T, hq, hkv, d = spec.total_tokens, spec.hq, spec.hkv, spec.head_dim
    if rank == 0:
        peaks = measured_peaks()
        kb = statistics.mean(kern_b)
        kf = statistics.mean(kern_f)
        kq = statistics.mean(kern_q)
        # Dominant kernel: the backward dK/dV kernel.  Algorithmic work per launch: the four GEMMs of
        # the dK/dV gradient it owns (S, dP, dV, dK = 8 d flops per causal pair per query head).
        fa = fb * 8 // 10
        ach = fa / (kb * 1e-3) / 1e12
        traffic = read_traffic("k_attn_bwd_dkdv", args)
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"config {args.config}: {spec.name} pool, {spec.n_seqs} x {spec.seq_len} tokens, "
                                   f"{len(lengths)} samples (log-normal median 644, sigma 1.6), Hq {hq} / Hkv {hkv} / d {d}, "
                                   f"causal per sample, fwd+bwd; plan built once and reused",
                       "tile_q": 256, "tile_kv": 128, "n_workers": plan.info()["n_workers"],
                       "tile_weight": "blocks (time proxy)" if args.weight_model == "blocks" else "causal pairs (Eq. 6)",
                       "l2": "inputs larger than L2 (Q alone is %.2f GB)" % (q.numel() * 2 / 1e9),
                       "per_rank_pool": "seed = rank"},
            "pct_of_bf16_peak": {"burst_measured": round(100 * value / world / peaks["burst"], 2),
                                 "sustained_measured": round(100 * value / world / peaks["sustained"], 2),
                                 "nominal_2250": round(100 * value / world / 2250.0, 2), "peaks": peaks["source"]},
            "fwd_kernel": {"ms": round(kf, 4), "tflops": round(ff / kf / 1e9, 1)},
            "bwd_dkdv_kernel": {"ms": round(kb, 4), "executed_tflops": round(fa / kb / 1e9, 1)},
            "bwd_dq_kernel": {"ms": round(kq, 4), "executed_tflops": round(fb * 6 // 10 / kq / 1e9, 1)},
            "bwd_useful_tflops": round(fb / (kb + kq) / 1e9, 1),
            "busy_max_over_mean": {"fwd": round(float(busy_f.max() / busy_f.mean()), 4),
                                   "bwd_dkdv": round(float(busy_b.max() / busy_b.mean()), 4),
                                   "bwd_dq": round(float(busy_q.max() / busy_q.mean()), 4)},
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": int(launches),
            "plan_ms": None if plan_ms is None else round(plan_ms, 3),
            "other_tile_weight": alt,
            "roofline": {"bound": "tensor", "kernel": "k_attn_bwd_dkdv", "achieved": round(ach, 1),
                         "peak": peaks["sustained"], "unit": "TFLOP/s", "frac": round(ach / peaks["sustained"], 4),
                         "peak_kind": f"bf16 sustained, {peaks['source']}", "traffic": traffic,
                         "frac_of_burst": round(ach / peaks["burst"], 4)},
        }
        if world == 1 and not args.skip_cpu:
            cb = time_oracle(spec, lengths)
            line["cpu_baseline"] = {k2: (round(v2, 6) if isinstance(v2, float) else v2) for k2, v2 in cb.items()}
        print(json.dumps(line), flush=True)


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
    ap.add_argument("--seqs", type=int, default=0, help="override the number of packed sequences (profiling runs)")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU oracle leg (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
