"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing and the whole-job
aggregation used for N > 1 replicas (the FFN path itself has no data-path collective)."""
import os
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch
    import bench
    rank, world, local = bench.dist_setup(2, backend="gloo")
    assert world == 2 and rank in (0, 1)
    bench.barrier(world, cuda=False)
    ms = 10.0 if rank == 0 else 30.0           # rank 1 is the slow replica
    ms_max = bench.max_over_ranks(ms, world, torch.device("cpu"))
    us = bench.whole_job_us_per_call(ms_max, steps=3, calls_per_step=1000, world=world)
    bench.barrier(world, cuda=False)
    if rank == 0:
        print(json.dumps({"ms_max": ms_max, "us": us}))
    import torch.distributed as dist
    dist.destroy_process_group()
""") % str(ROOT)


def test_two_gloo_ranks_take_the_slowest_time_and_aggregate_the_job(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = []
    for r in range(2):
        procs.append(subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json

    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["ms_max"] == 30.0                              # the slowest rank decides
    assert abs(res["us"] - 30.0 * 1e3 / (3 * 1000 * 2)) < 1e-9  # two replicas did twice the calls


def test_single_process_defaults():
    sys.path.insert(0, str(ROOT))
    import bench

    assert bench.max_over_ranks(5.0, 1, None) == 5.0
    assert bench.whole_job_us_per_call(31.0, 1, 1000, 1) == 31.0
    peak, kind = bench.measured_hbm_peak()
    assert peak > 1000 and kind in ("measured", "fallback")
