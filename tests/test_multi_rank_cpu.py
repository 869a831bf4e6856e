"""The N>1 launch contract of bench.py on CPU: two gloo ranks, replicas with no data-path
collective, time = max over ranks, whole-job value = N x per-rank units / that time, and the
reference arm prints on rank 0 only."""
import json
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
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    bench.barrier(world)
    ms_local = 10.0 + 5.0 * rank                    # rank 1 is the slow replica
    value, ms = bench.aggregate_throughput(1000, ms_local, world, torch.device("cpu"))
    m = bench.max_over_ranks(float(rank), world, torch.device("cpu"))
    bench.barrier(world)
    if rank == 0:
        print(json.dumps({"value": value, "ms": ms, "max": m, "world": world}), flush=True)
    dist.destroy_process_group()
""" % ROOT)


def test_two_gloo_ranks_aggregate_like_the_bench(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                           # only rank 0 reports
    d = json.loads(lines[0])
    assert d["world"] == 2 and d["max"] == 1.0
    assert abs(d["ms"] - 15.0) < 1e-9                # the slowest rank sets the time
    assert abs(d["value"] - 2 * 1000 / 15e-3) < 1e-6


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=120, env=env, cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == ""
