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


def test_clock_sampler_reads_clocks_power_and_reasons(tmp_path, monkeypatch):
    """The bench's clock record comes from nvidia-smi's csv lines; a stand-in on PATH prints three samples."""
    import stat
    import time
    fake = tmp_path / "nvidia-smi"
    fake.write_text("#!/bin/sh\n"
                    "echo '1200, 1965, 990.5, Not Active, Not Active, Not Active, Active'\n"
                    "echo '1100, 1965, 1001.0, Not Active, Not Active, Not Active, Active'\n"
                    "echo '1300, 1965, [N/A], Not Active, Not Active, Not Active, Not Active'\n"
                    "sleep 30\n")
    fake.chmod(fake.stat().st_mode | stat.S_IEXEC)
    monkeypatch.setenv("PATH", str(tmp_path) + os.pathsep + os.environ["PATH"])
    sys.path.insert(0, ROOT)
    import bench
    s = bench.ClockSampler(0)
    s.start()
    time.sleep(0.5)
    rec = s.stop()
    assert rec["samples"] == 3 and rec["sm_mhz"] == 1200 and rec["sm_max_mhz"] == 1965
    assert rec["reasons"] == ["sw_power_cap"]
    assert rec["power_w"] == (990.5 + 1001.0) / 2          # the unreadable sample is left out
