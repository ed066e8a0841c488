"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, each with its own shard of the workload,
agree on the job's step time (max over ranks) and on the aggregate value.  No GPU, no data-path collective."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2607_12789_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = bench.shard_workload(synth.C0, rank)
    x = synth.generate(wl)
    my_ms = 1.0 + 0.5 * rank                                   # rank 1 is the slow one
    ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    dist.barrier()
    out[rank] = (wl.seed, float(x["K"].sum()), ms, bench.job_value(synth.C0, world, ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_share_nothing_but_the_step_time():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] != r1[0] and r0[1] != r1[1]                   # different seeds, different data
    assert r0[2] == r1[2] == 1.5                               # both see the slowest rank's time
    assert r0[3] == r1[3] == 2 * 1 * 256 / 1.5e-3              # tokens of both ranks over that time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(2.5, 1, torch.device("cpu")) == 2.5


def test_timed_loop_is_repeated_until_enough_time_is_covered():
    import bench
    assert bench.repeats_for(5.6) == 36                        # 20 steps of 0.28 ms: 36 repeats reach 200 ms
    assert bench.repeats_for(500.0) == 1
    assert bench.repeats_for(1e-4) == bench.MAX_REPEATS


def test_recorded_dram_traffic_is_dropped_when_the_kernel_sources_changed(tmp_path, monkeypatch):
    import json
    import bench
    from paper_2607_12789_b200 import build
    prof = tmp_path / "profiles"
    prof.mkdir()
    rec = dict(source_hash=build.source_hash(), command="ncu ...",
               entries=[dict(workload="c3_long", kernel="attend", dram_bytes_per_launch=1.0e8)])
    (prof / "ncu_traffic.json").write_text(json.dumps(rec))
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.measured_traffic("c3_long", "attend")[0] == 1.0e8
    assert bench.measured_traffic("c1_vitb", "attend")[0] is None
    rec["source_hash"] = "0" * 16
    (prof / "ncu_traffic.json").write_text(json.dumps(rec))
    assert bench.measured_traffic("c3_long", "attend")[0] is None
