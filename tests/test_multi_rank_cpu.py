"""The N > 1 path of bench.py is "replicas only": every rank runs the same single-GPU workload and
the timings are combined as max over ranks.  These tests run that host-side logic with two gloo
ranks on CPU (no GPU, no NCCL)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    rank, world, local = bench.dist_setup(int(os.environ["WORLD_SIZE"]))
    dist.init_process_group("gloo")
    # every rank "measured" a different time; the job's time is the slowest rank's
    mine = 10.0 + 5.0 * rank
    mx = bench.max_over_ranks(mine, world, None)
    value = bench.aggregate_value(6.0e12, 4, world, mx)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"rank": rank, "world": world, "max_ms": mx, "value": value}))
    dist.destroy_process_group()
""") % ROOT


def _spawn(world, port):
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    return outs


def test_two_gloo_ranks_aggregate_as_replicas():
    import json
    outs = _spawn(2, 29731)
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["world"] == 2 and line["max_ms"] == 15.0
    # whole-job value: both ranks' work over the slowest rank's time
    assert abs(line["value"] - 6.0e12 * 4 * 2 / 15.0e-3 / 1e12) < 1e-6
    assert outs[1][0].strip() == ""          # only rank 0 prints


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.flops_per_step(16384, 8192, 8192) == 6.0 * 16384 * 8192 * 8192
    assert abs(bench.aggregate_value(1e12, 10, 1, 10.0) - 1000.0) < 1e-9
