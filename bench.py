#!/usr/bin/env python
"""Benchmark of the AVQ-attention forward (assign -> aggregate -> attend) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c2|c3|N4096_M128_P16]
    python bench.py --impl reference ...       # the fp64 CPU oracle on the host cores

One "step" is one avq_forward call over one batch of seeded synthetic inputs (every stage
of the path).  Prints ONE JSON line:

  value            query-tokens/s (B*Nq / t, summed over GPUs), inputs resident in HBM
  e2e              the same through avq_forward_host: pinned host Q,K,V -> device, forward, Y -> host
  roofline         the dominant stage's kernel against the measured HBM / tensor peak
  forward_roofline the whole call against max(attention FLOPs / tensor peak, Q+K+V+Y bytes / HBM peak)
  cpu_baseline     the oracle timed on a bounded sample of the same workload on this host
  also             the same headline numbers for the other large configurations

Inputs rotate through enough independent copies that their footprint exceeds twice the L2,
so no step finds its inputs cached.  With N > 1 (torchrun) every rank runs its own batch
(weak scaling); no collective touches the data path, only the barrier and the max-over-ranks
of the step time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "avq_attn_fwd_query_tokens_per_s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of each stage's kernel(s), from the ncu captures
# summarised under profiles/ (tc_attend_c1.md, tc_attend_c3.md, tc_assign_c3.md, kernels_c2_and_N16384_M64_P8.md);
# other workloads: None.
NCU_TRAFFIC = {
    ("c1_vitb", "assign"): 13.12e6, ("c1_vitb", "aggregate"): 17.67e6 + 6.40e6, ("c1_vitb", "attend"): 14.80e6,
    ("c2_mid", "assign"): 19.06e6, ("c2_mid", "aggregate"): 22.55e6 + 8.54e6, ("c2_mid", "attend"): 19.19e6,
    ("c3_long", "assign"): 71.58e6 + 2.68e6, ("c3_long", "aggregate"): 75.16e6 + 0.92e6 + 8.46e6,
    ("c3_long", "attend"): 71.52e6 + 25.32e6,
}
UNIT = "query-tokens/s"


def parse_workload(name: str):
    from paper_2607_12789_b200 import synth
    if name in synth.NAMED:
        return synth.NAMED[name]
    try:
        parts = dict((p[0], int(p[1:])) for p in name.split("_"))
        return synth.sweep_point(parts["N"], parts["M"], parts["P"])
    except Exception as e:  # pragma: no cover
        raise SystemExit(f"unknown workload {name!r}: {e}")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), tflops=float(p["bf16_tflops"]),
                    tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, tflops=1590.0, tflops_sustained=1400.0, source="fallback")


def model(wl):
    """Algorithmic bytes and flops of one forward and of each stage (per GPU)."""
    es = 4 if wl.dtype == "f32" else 2
    BH, N, d, M, C, P = wl.B * wl.H, wl.N, wl.d, wl.M, wl.C, wl.P
    tens = BH * N * d * es
    agg_f32 = BH * M * (1 + C) * (d + 1) * 4
    agg_b16 = BH * M * (1 + C) * d * 2
    books = wl.H * M * (1 + C) * d * es
    st = {
        "assign": dict(bytes=tens + BH * N * 8 + books, flops=2.0 * BH * N * (M + C) * d),
        "aggregate": dict(bytes=tens + BH * N * 8 + 2 * agg_f32 + agg_b16, flops=2.0 * BH * N * d),
        "attend": dict(bytes=2 * tens + agg_b16 + BH * M * (1 + C) * 4 + books,
                       flops=2.0 * BH * N * (M + P * C) * d * 2),
    }
    fwd = dict(bytes=4 * tens, flops=2.0 * BH * N * (M + P * C) * d * 2)
    return st, fwd


def roof(entry, pk, ms, dtype):
    tflops_peak = pk["tflops"] if dtype == "bf16" else pk["tflops"] / 16.0   # fp32 path runs on CUDA cores
    t_hbm = entry["bytes"] / (pk["hbm_gbs"] * 1e9)
    t_tc = entry["flops"] / (tflops_peak * 1e12)
    if t_hbm >= t_tc:
        ach = entry["bytes"] / (ms * 1e-3) / 1e9
        return dict(bound="hbm", achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"])
    ach = entry["flops"] / (ms * 1e-3) / 1e12
    return dict(bound="tensor", achieved=ach, peak=tflops_peak, unit="TFLOP/s", frac=ach / tflops_peak)


def shard_workload(wl, rank: int):
    """Weak scaling: every rank runs its own batch of the same shape (its own seed), no data exchange."""
    return wl.with_(seed=wl.seed + 7919 * rank)


def max_over_ranks(ms: float, world: int, device) -> float:
    """Step time of the job = the slowest rank's (one MAX all-reduce of a scalar; nothing else is exchanged)."""
    if world <= 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def job_value(wl, world: int, ms: float) -> float:
    """Query tokens per second of the whole job (all ranks)."""
    return wl.B * wl.N * world / (ms * 1e-3)


class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except Exception:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons),
                    window="warm-up, timed steps and 1 s more of the same step")


def run_gpu(wl, steps, warmup, rank, world, flags=0, extras=True, min_warm_s=0.3, spin=True):
    import torch
    from paper_2607_12789_b200 import binding, synth
    dev = torch.device("cuda", torch.cuda.current_device())
    td = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    x = synth.generate(shard_workload(wl, rank))
    host = {k: torch.from_numpy(v).to(td) for k, v in x.items()}
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    foot = sum(host[k].numel() * host[k].element_size() for k in "QKV") + host["Q"].numel() * host["Q"].element_size()
    copies = max(2, math.ceil(2.0 * l2 / foot))
    sets = []
    for _ in range(copies):
        s = {k: host[k].to(dev) for k in "QKV"}
        s["Y"] = torch.empty_like(s["Q"])
        sets.append(s)
    Cp, Cc = host["Cp"].to(dev), host["Cc"].to(dev)
    f = binding.Forward(wl.B, wl.H, wl.N, wl.N, wl.d, wl.M, wl.C, wl.P, wl.block_q, dtype=td, scale=wl.scale,
                        flags=flags, device=dev)

    def step(i):
        s = sets[i % copies]
        f(s["Q"], s["K"], s["V"], Cp, Cc, s["Y"])

    def timed(fn, n, head_start=True):
        # Device time between two events.  A spin kernel queued first keeps the GPU busy while the host
        # enqueues the calls, so that short kernels are not timed at the host's enqueue rate; the
        # end-to-end loop (whose host work is part of what is measured) runs without it.
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if head_start and spin:
            torch.cuda._sleep(int(2.0e6 * min(n, 64) / 10))
        e0.record()
        for i in range(n):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    def barrier():
        if world > 1:
            torch.distributed.barrier()

    sampler = ClockSampler(dev.index) if extras else None
    t_end = time.time() + min_warm_s
    i = 0
    while i < max(3, warmup) or time.time() < t_end:
        step(i)
        i += 1
    torch.cuda.synchronize()
    f.check()
    barrier()
    ms = timed(step, steps)
    barrier()
    ms = max_over_ranks(ms, world, dev)
    f.check()
    out = dict(ms=ms, copies=copies, footprint_mb=foot * copies / 1e6, l2_mb=l2 / 1e6)
    if not extras:
        return out

    # sustained second of the same step, only so that the clock samples are taken under this load
    t_end = time.time() + 1.0
    while time.time() < t_end:
        for i in range(50):
            step(i)
        torch.cuda.synchronize()
    out["clocks"] = sampler.stop()

    # per-stage device times (same rotation), for the roofline of the dominant kernel
    pidx = torch.empty((wl.B, wl.H, wl.N), dtype=torch.int32, device=dev)
    cidx = torch.empty_like(pidx)
    f32 = dict(dtype=torch.float32, device=dev)
    Vp, n_p = torch.empty((wl.B, wl.H, wl.M, wl.d), **f32), torch.empty((wl.B, wl.H, wl.M), **f32)
    Vc, n_c = torch.empty((wl.B, wl.H, wl.M, wl.C, wl.d), **f32), torch.empty((wl.B, wl.H, wl.M, wl.C), **f32)
    import ctypes
    L, prob, st_ = binding.lib(), f.prob, binding._stream
    P_ = binding._ptr

    def s_assign(i):
        L.avq_assign(ctypes.byref(prob), P_(sets[i % copies]["K"]), P_(Cp), P_(Cc), P_(pidx), P_(cidx), st_())

    def s_aggregate(i):
        L.avq_aggregate(ctypes.byref(prob), P_(sets[i % copies]["V"]), P_(pidx), P_(cidx), P_(Vp), P_(n_p), P_(Vc),
                        P_(n_c), st_())

    def s_attend(i):
        s = sets[i % copies]
        f.attend(s["Q"], Cp, Cc, s["Y"])

    n_stage = max(steps, 20)
    s_assign(0)
    stages = {}
    for name, fn in (("assign", s_assign), ("aggregate", s_aggregate), ("attend", s_attend)):
        for i in range(3):
            fn(i)
        stages[name] = timed(fn, n_stage)
    out["stages_ms"] = stages

    # end to end: pinned host Q, K, V -> device, forward, Y -> pinned host, every step
    hq, hk, hv = (host[k].pin_memory() for k in "QKV")
    hy = torch.empty_like(hq).pin_memory()
    s0 = sets[0]
    e2e_fn = lambda i: f.host(hq, hk, hv, Cp, Cc, hy, s0["Q"], s0["K"], s0["V"], s0["Y"])
    for i in range(3):
        e2e_fn(i)
    barrier()
    e2e_ms = timed(e2e_fn, steps, head_start=False)
    barrier()
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    f.check()
    es = hq.element_size()
    out["e2e"] = dict(ms=e2e_ms, h2d=3 * hq.numel() * es, d2h=hq.numel() * es,
                      y_checksum=float(hy.float().abs().mean()))
    return out


def oracle_sample(wl, budget_s, steps_total=1):
    """Times the oracle (dense form, as it stands) on whole heads of the workload.  Returns
    (seconds per step, heads per step, threads)."""
    from oracle import avq_oracle as orc
    from paper_2607_12789_b200 import synth
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = 1
    small = wl.with_(B=1, H=min(wl.H, 4))
    x = synth.generate(small)

    def head(i):
        h = i % small.H
        orc.forward_head(x["Q"][0, h], x["K"][0, h], x["V"][0, h], x["Cp"][h], x["Cc"][h], wl.P, wl.block_q,
                         wl.scale, form="dense")

    t0 = time.time()
    head(0)
    t_head = time.time() - t0
    heads = int(max(1, min(wl.B * wl.H, budget_s / max(t_head, 1e-3) / steps_total)))
    return head, heads, t_head, cores


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c1")
    ap.add_argument("--also", default="c2,c3", help="comma list of further workloads reported under 'also'")
    ap.add_argument("--simt", action="store_true", help="force the CUDA-core kernels (cross-check)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every (N, M, P) point of the sweep configuration; one JSON line per point")
    ap.add_argument("--profile", action="store_true",
                    help="only W warm-up and K timed steps (no stage timing, e2e, CPU baseline): for ncu")
    args = ap.parse_args()
    wl = parse_workload(args.workload)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    warm = max(3, args.warmup)
    stage_model, fwd_model = model(wl)
    config = dict(workload=wl.name, B=wl.B, H=wl.H, N=wl.N, d=wl.d, M=wl.M, C=wl.C, P=wl.P, block_q=wl.block_q,
                  logit_scale="1/sqrt(d)", per_gpu_batch=wl.B)

    if args.impl == "reference":
        if rank != 0:
            return
        head, heads, t_head, cores = oracle_sample(wl, budget_s=150.0, steps_total=args.steps + warm)
        for _ in range(warm):
            for i in range(heads):
                head(i)
        t0 = time.time()
        for _ in range(args.steps):
            for i in range(heads):
                head(i)
        dt = (time.time() - t0) / args.steps
        val = heads * wl.N / wl.H / dt
        sample = f"{heads} of {wl.B * wl.H} (batch, head) pairs per step, dense O(N^2) form, fp64"
        print(json.dumps(dict(impl="reference", metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus,
                              steps=args.steps, warmup=warm, ms_per_step=dt * 1e3, higher_is_better=True,
                              scaling="weak", vs_baseline=None, dtype="f64", data="synthetic", config=config,
                              cpu_baseline=dict(value=val, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                              e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local))
    flags = 2 if args.simt else 0
    pk = peaks()
    if args.sweep:
        from paper_2607_12789_b200 import synth
        for N in synth.SWEEP_N:
            for M in synth.SWEEP_M:
                for P in synth.sweep_P(M):
                    w2 = synth.sweep_point(N, M, P)
                    r2 = run_gpu(w2, max(5, args.steps // 5), 3, 0, 1, flags=flags, extras=False, min_warm_s=0.0)
                    _, f2 = model(w2)
                    fr2 = roof(f2, pk, r2["ms"], w2.dtype)
                    print(json.dumps(dict(workload=w2.name, N=N, M=M, P=P, ms_per_step=r2["ms"],
                                          value=w2.B * w2.N / (r2["ms"] * 1e-3), unit=UNIT,
                                          tflops=f2["flops"] / (r2["ms"] * 1e-3) / 1e12, bound=fr2["bound"],
                                          forward_roofline_frac=fr2["frac"])), flush=True)
        return
    if args.profile:
        res = run_gpu(wl, args.steps, warm, rank, world, flags=flags, extras=False, min_warm_s=0.0, spin=False)
        if rank == 0:
            print(json.dumps(dict(metric=METRIC, profile_only=True, ms_per_step=res["ms"], config=config)))
        return
    res = run_gpu(wl, args.steps, warm, rank, world, flags=flags)
    ms = res["ms"]
    tokens = wl.B * wl.N * world
    value = job_value(wl, world, ms)
    dom = max(res["stages_ms"], key=res["stages_ms"].get)
    rl = roof(stage_model[dom], pk, res["stages_ms"][dom], wl.dtype)
    rl.update(kernel=dom, traffic=NCU_TRAFFIC.get((wl.name, dom)), peak_source=pk["source"],
              bytes_per_launch=stage_model[dom]["bytes"], flops_per_launch=stage_model[dom]["flops"],
              ms_per_launch=res["stages_ms"][dom])
    fr = roof(fwd_model, pk, ms, wl.dtype)
    fr.update(tflops=fwd_model["flops"] / (ms * 1e-3) / 1e12, gbs=fwd_model["bytes"] / (ms * 1e-3) / 1e9,
              roofline_us=max(fwd_model["bytes"] / (pk["hbm_gbs"] * 1e9),
                              fwd_model["flops"] / (pk["tflops"] * 1e12)) * 1e6)
    stages = {k: dict(ms=v, **{kk: vv for kk, vv in roof(stage_model[k], pk, v, wl.dtype).items()
                              if kk in ("bound", "frac")}) for k, v in res["stages_ms"].items()}
    e2e_val = tokens / (res["e2e"]["ms"] * 1e-3)
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warm, ms_per_step=ms,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype=wl.dtype, data="synthetic",
                config=dict(config, l2_policy=f"inputs rotate through {res['copies']} copies "
                                             f"({res['footprint_mb']:.0f} MB > 2 x L2 {res['l2_mb']:.0f} MB)",
                            kernels="cuda-core" if (args.simt or wl.dtype == "f32") else "tcgen05"),
                clocks=res["clocks"],
                e2e=dict(value=e2e_val, unit=UNIT, ms_per_step=res["e2e"]["ms"],
                         h2d_bytes_per_step=res["e2e"]["h2d"], d2h_bytes_per_step=res["e2e"]["d2h"]),
                gpu_launches=4 * args.steps, roofline=rl, forward_roofline=fr, stages=stages)

    if rank == 0 and args.also and world == 1:
        also = []
        for name in [a for a in args.also.split(",") if a and a != args.workload]:
            w2 = parse_workload(name)
            r2 = run_gpu(w2, max(10, args.steps // 2), 5, 0, 1, flags=flags, extras=False)
            _, f2 = model(w2)
            fr2 = roof(f2, pk, r2["ms"], w2.dtype)
            also.append(dict(workload=w2.name, value=w2.B * w2.N / (r2["ms"] * 1e-3), unit=UNIT, ms_per_step=r2["ms"],
                             tflops=f2["flops"] / (r2["ms"] * 1e-3) / 1e12, forward_roofline_frac=fr2["frac"],
                             bound=fr2["bound"]))
        line["also"] = also

    if rank == 0 and world == 1:
        head, heads, t_head, cores = oracle_sample(wl, budget_s=12.0)
        t0, done = time.time(), 0
        while done == 0 or time.time() - t0 < 10.0:
            for i in range(heads):
                head(i)
            done += heads
        dt = time.time() - t0
        line["cpu_baseline"] = dict(value=done * wl.N / wl.H / dt, unit=UNIT, cores=cores, kind="oracle",
                                    sample=f"{done} (batch, head) problems of this workload's shape "
                                           f"({wl.B * wl.H} make one step), dense O(N^2) form, fp64, {dt:.1f} s")
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
