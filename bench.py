#!/usr/bin/env python
"""Benchmark of the AVQ-attention forward (assign -> aggregate -> attend) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c1|N4096_M128_P16]
    python bench.py --impl reference ...       # the fp64 CPU oracle on the host cores

One "step" is one avq_forward call over one batch of seeded synthetic inputs (every stage
of the path).  The default workload is the largest single-GPU configuration (c3: B1 H16
N16384 d128 M256 C4 P32); the other large ones are reported under `also`.  Prints ONE JSON line:

  value            query-tokens/s (B*Nq / t, summed over GPUs), inputs resident in HBM
  e2e              the same through avq_forward_host: pinned host Q,K,V -> device, forward, Y -> host
  roofline         the dominant stage's kernel against the measured HBM / tensor peak
  forward_roofline the whole call against max(attention FLOPs / tensor peak, Q+K+V+Y bytes / HBM peak)
  cpu_baseline     the oracle timed on a bounded sample of the same workload on this host
  also             the same numbers (own clock window, stages, dominant kernel) for the other workloads

Timing: W warm-up steps, then the K-step loop is timed with CUDA events on the launching stream and
repeated until at least 200 ms have been timed; `ms_per_step` is the median of the repeats (the minimum
is reported beside it).  Inputs rotate through enough independent copies that their footprint exceeds
twice the L2, so no step finds its inputs cached.  With N > 1 every rank runs its own batch (weak
scaling); no collective touches the data path, only the barrier and the max-over-ranks of the step
time.  `--gpus N` without a torchrun environment starts the N local ranks itself.
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
UNIT = "query-tokens/s"
MIN_TIMED_MS = 200.0
MAX_REPEATS = 200
L2_POLICY = "inputs rotate through independent copies whose total footprint exceeds twice the L2"
# Datasheet figures (HGX B200: HBM3e 7.7 TB/s, dense bf16 2.25 PFLOP/s), printed beside the measured peaks.
NOMINAL = dict(hbm_gbs=7700.0, tflops=2250.0)
KERNELS_PER_STEP = 5          # codeword norms, assign, leaf scatter, finalize, attend


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


def measured_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of a stage's kernels from the last ncu capture, or None when the capture was
    taken from other kernel sources than the ones this run was built from."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return None, "no capture recorded"
    from paper_2607_12789_b200 import build
    rec = json.load(open(path))
    if rec.get("source_hash") != build.source_hash():
        return None, "kernel sources changed since the capture"
    for e in rec.get("entries", []):
        if e["workload"] == workload and e["kernel"] == kernel:
            return float(e["dram_bytes_per_launch"]), rec.get("command", "")
    return None, "workload not captured"


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
    scale = 1.0 if dtype == "bf16" else 1.0 / 16.0          # the fp32 path runs on CUDA cores
    tflops_peak = pk["tflops"] * scale
    t_hbm = entry["bytes"] / (pk["hbm_gbs"] * 1e9)
    t_tc = entry["flops"] / (tflops_peak * 1e12)
    if t_hbm >= t_tc:
        ach = entry["bytes"] / (ms * 1e-3) / 1e9
        return dict(bound="hbm", achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"],
                    frac_nominal=ach / NOMINAL["hbm_gbs"])
    ach = entry["flops"] / (ms * 1e-3) / 1e12
    return dict(bound="tensor", achieved=ach, peak=tflops_peak, unit="TFLOP/s", frac=ach / tflops_peak,
                frac_nominal=ach / (NOMINAL["tflops"] * scale))


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


def repeats_for(first_loop_ms: float) -> int:
    """How many times the K-step loop is timed in all (the first one included): enough for MIN_TIMED_MS."""
    return int(min(MAX_REPEATS, max(1, math.ceil(MIN_TIMED_MS / max(first_loop_ms, 1e-6)))))


def launch_local_ranks(n: int, argv) -> int:
    """`--gpus N` without a torchrun environment: start the N ranks of this node ourselves."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


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
                    window="warm-up, the timed repeats and 1 s more of the same step")


def run_gpu(wl, steps, warmup, rank, world, flags=0, clocks=True, stages=True, e2e=True, repeat=True,
            min_warm_s=0.3, spin=True):
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

    def timed_once(fn, n, head_start=True):
        # Device time between two events on the launching stream.  A spin kernel queued first keeps the
        # GPU busy while the host enqueues the calls, so that short kernels are not timed at the host's
        # enqueue rate; the end-to-end loop (whose host work is part of what is measured) runs without it.
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

    def timed(fn, n, head_start=True, collective=True):
        """Median and minimum per-step time over repeats of the n-step loop (>= MIN_TIMED_MS timed in all)."""
        if collective:
            barrier()
        first = timed_once(fn, n, head_start)
        if collective:
            barrier()
            first = max_over_ranks(first, world, dev)
        runs = [first]
        reps = repeats_for(first * n) if repeat else 1
        for _ in range(reps - 1):
            if collective:
                barrier()
            t = timed_once(fn, n, head_start)
            if collective:
                barrier()
                t = max_over_ranks(t, world, dev)
            runs.append(t)
        return dict(ms=statistics.median(runs), ms_min=min(runs), repeats=len(runs))

    sampler = ClockSampler(dev.index) if clocks else None
    t_end = time.time() + min_warm_s
    i = 0
    while i < max(3, warmup) or time.time() < t_end:
        step(i)
        i += 1
    torch.cuda.synchronize()
    f.check()
    r = timed(step, steps)
    f.check()
    out = dict(ms=r["ms"], ms_min=r["ms_min"], repeats=r["repeats"], copies=copies,
               footprint_mb=foot * copies / 1e6, l2_mb=l2 / 1e6)

    if clocks:
        # one more second of the same step, so that the clock samples are taken under this load
        t_end = time.time() + 1.0
        while time.time() < t_end:
            for i in range(20):
                step(i)
            torch.cuda.synchronize()
        out["clocks"] = sampler.stop()

    if stages:
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
            L.avq_aggregate(ctypes.byref(prob), P_(sets[i % copies]["V"]), P_(pidx), P_(cidx), P_(Vp), P_(n_p),
                            P_(Vc), P_(n_c), st_())

        def s_attend(i):
            s = sets[i % copies]
            f.attend(s["Q"], Cp, Cc, s["Y"])

        s_assign(0)
        res = {}
        for name, fn in (("assign", s_assign), ("aggregate", s_aggregate), ("attend", s_attend)):
            for i in range(3):
                fn(i)
            res[name] = timed(fn, max(steps, 10), collective=False)["ms"]
        f.check()
        out["stages_ms"] = res

    if e2e:
        # end to end: pinned host Q, K, V -> device, forward, Y -> pinned host, every step
        hq, hk, hv = (host[k].pin_memory() for k in "QKV")
        hy = torch.empty_like(hq).pin_memory()
        s0 = sets[0]
        e2e_fn = lambda i: f.host(hq, hk, hv, Cp, Cc, hy, s0["Q"], s0["K"], s0["V"], s0["Y"])
        for i in range(3):
            e2e_fn(i)
        r = timed(e2e_fn, steps, head_start=False)
        f.check()
        es = hq.element_size()
        out["e2e"] = dict(ms=r["ms"], ms_min=r["ms_min"], repeats=r["repeats"], h2d=3 * hq.numel() * es,
                          d2h=hq.numel() * es, y_checksum=float(hy.float().abs().mean()))
    return out


def oracle_sample(wl, budget_s, steps_total=1):
    """The oracle (dense form, as it stands) on whole (batch, head) problems of the workload.  Returns
    (callable running problem i, problems per step, seconds for one problem, threads)."""
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


def describe(wl, res, pk, steps, world):
    """The numbers of one workload: throughput, whole-forward roofline, stages, dominant kernel."""
    stage_model, fwd_model = model(wl)
    ms = res["ms"]
    d = dict(value=job_value(wl, world, ms), unit=UNIT, ms_per_step=ms, ms_per_step_min=res["ms_min"],
             repeats=res["repeats"])
    fr = roof(fwd_model, pk, ms, wl.dtype)
    fr.update(tflops=fwd_model["flops"] / (ms * 1e-3) / 1e12, gbs=fwd_model["bytes"] / (ms * 1e-3) / 1e9,
              roofline_us=max(fwd_model["bytes"] / (pk["hbm_gbs"] * 1e9),
                              fwd_model["flops"] / (pk["tflops"] * 1e12)) * 1e6, peak_source=pk["source"])
    d["forward_roofline"] = fr
    if "stages_ms" in res:
        dom = max(res["stages_ms"], key=res["stages_ms"].get)
        rl = roof(stage_model[dom], pk, res["stages_ms"][dom], wl.dtype)
        traffic, note = measured_traffic(wl.name, dom)
        rl.update(kernel=dom, traffic=traffic, traffic_source=note, peak_source=pk["source"],
                  bytes_per_launch=stage_model[dom]["bytes"], flops_per_launch=stage_model[dom]["flops"],
                  ms_per_launch=res["stages_ms"][dom])
        d["roofline"] = rl
        d["stages"] = {k: dict(ms=v, **{kk: vv for kk, vv in roof(stage_model[k], pk, v, wl.dtype).items()
                                       if kk in ("bound", "frac", "frac_nominal")})
                       for k, v in res["stages_ms"].items()}
    if "clocks" in res:
        d["clocks"] = res["clocks"]
    return d


def config_of(wl):
    return dict(workload=wl.name, B=wl.B, H=wl.H, N=wl.N, d=wl.d, M=wl.M, C=wl.C, P=wl.P, block_q=wl.block_q,
                logit_scale="1/sqrt(d)", per_gpu_batch=wl.B, l2_policy=L2_POLICY)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--also", default="c2,c1", help="comma list of further workloads reported under 'also'")
    ap.add_argument("--simt", action="store_true", help="force the CUDA-core kernels (cross-check)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every (N, M, P) point of the sweep configuration; one JSON line per point")
    ap.add_argument("--profile", action="store_true",
                    help="only W warm-up and K timed steps (no repeats, stage timing, e2e, CPU baseline): for ncu")
    args = ap.parse_args()
    wl = parse_workload(args.workload)
    in_torchrun = "WORLD_SIZE" in os.environ
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and not in_torchrun:
        if args.impl == "reference":
            world = 1                      # the CPU oracle runs once, on this process
        else:
            sys.exit(launch_local_ranks(args.gpus, sys.argv[1:]))
    if in_torchrun and args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE {world}")
    warm = max(3, args.warmup)
    config = config_of(wl)

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
                    r2 = run_gpu(w2, max(5, args.steps // 2), 3, 0, 1, flags=flags, clocks=False, stages=False,
                                 e2e=False, min_warm_s=0.0)
                    _, f2 = model(w2)
                    fr2 = roof(f2, pk, r2["ms"], w2.dtype)
                    print(json.dumps(dict(workload=w2.name, N=N, M=M, P=P, ms_per_step=r2["ms"],
                                          ms_per_step_min=r2["ms_min"], repeats=r2["repeats"],
                                          value=w2.B * w2.N / (r2["ms"] * 1e-3), unit=UNIT,
                                          tflops=f2["flops"] / (r2["ms"] * 1e-3) / 1e12, bound=fr2["bound"],
                                          forward_roofline_frac=fr2["frac"])), flush=True)
        return
    if args.profile:
        res = run_gpu(wl, args.steps, warm, rank, world, flags=flags, clocks=False, stages=False, e2e=False,
                      repeat=False, min_warm_s=0.0, spin=False)
        if rank == 0:
            print(json.dumps(dict(metric=METRIC, profile_only=True, ms_per_step=res["ms"], config=config)))
        return

    res = run_gpu(wl, args.steps, warm, rank, world, flags=flags)
    d = describe(wl, res, pk, args.steps, world)
    tokens = wl.B * wl.N * world
    line = dict(metric=METRIC, value=d["value"], unit=UNIT, n_gpus=world, steps=args.steps, warmup=warm,
                ms_per_step=d["ms_per_step"], ms_per_step_min=d["ms_per_step_min"], repeats=d["repeats"],
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype=wl.dtype, data="synthetic",
                config=config, kernels="cuda-core" if (args.simt or wl.dtype == "f32") else "tcgen05",
                l2=dict(copies=res["copies"], footprint_mb=res["footprint_mb"], l2_mb=res["l2_mb"]),
                clocks=d["clocks"],
                e2e=dict(value=tokens / (res["e2e"]["ms"] * 1e-3), unit=UNIT, ms_per_step=res["e2e"]["ms"],
                         ms_per_step_min=res["e2e"]["ms_min"], repeats=res["e2e"]["repeats"],
                         h2d_bytes_per_step=res["e2e"]["h2d"], d2h_bytes_per_step=res["e2e"]["d2h"]),
                gpu_launches=KERNELS_PER_STEP * args.steps * d["repeats"], gpu_launches_per_step=KERNELS_PER_STEP,
                roofline=d["roofline"], forward_roofline=d["forward_roofline"], stages=d["stages"],
                nominal_peaks=NOMINAL)

    if rank == 0 and args.also and world == 1:
        also = []
        for name in [a for a in args.also.split(",") if a and parse_workload(a).name != wl.name]:
            w2 = parse_workload(name)
            r2 = run_gpu(w2, args.steps, warm, 0, 1, flags=flags, e2e=False)
            d2 = describe(w2, r2, pk, args.steps, 1)
            d2["workload"] = w2.name
            also.append(d2)
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
