"""Host-side logic of the benchmark that involves more than one process (replicas only:
the path has no exchange step, so N GPUs run N independent replicas and only timing is
reduced).  Runs on CPU with the gloo backend, world size 2."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
local_seconds = 2.0 if rank == 0 else 3.0          # rank 1 is the slow one
assert bench.max_over_ranks(local_seconds, dist) == 3.0
rate = bench.whole_job_rate(600, local_seconds, dist)
assert abs(rate - 2 * 600 / 3.0) < 1e-9, rate
assert bench.whole_job_rate(600, 2.0) == 300.0     # no process group: one replica
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_whole_job_rate_is_all_units_over_slowest_rank():
    port = free_port()
    code = WORKER.format(root=ROOT, port=port)
    procs = [subprocess.Popen([sys.executable, "-c", code, str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"ok {r}" in out


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--config", "1"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["higher_is_better"] is True


def test_gpus_flag_starts_the_replicas_itself():
    """`bench.py --gpus 2` outside a launcher re-executes itself under torchrun with two ranks
    (replicas only); the reference arm needs no GPU, so the whole launch runs here."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env["OMP_NUM_THREADS"] = "2"
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--config", "1"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2
    assert 0.0 <= d["cpu_baseline"]["sample_density"] <= 1.0


def test_repeat_plan_and_launch_command():
    sys.path.insert(0, ROOT)
    import bench
    # a 41 ms region (20 steps of the headline config) is repeated until 2 s have been timed
    assert bench.plan_repeats(0.041) == 49
    assert bench.plan_repeats(0.52) == 5 and bench.plan_repeats(10.0) == 5     # never fewer than five
    assert bench.plan_repeats(1e-5) == 200                                      # bounded
    assert bench.median([3.0, 1.0, 2.0]) == 2.0 and bench.median([4.0, 1.0, 2.0, 3.0]) == 2.5
    cmd = bench.replica_launch_command(4, ["--gpus", "4", "--steps", "20"], port=29512)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "20"] and cmd[-5].endswith("bench.py")
    # clock samples are attributed to a repeat by the time they were taken
    cs = bench.ClockSampler(0)
    cs.samples = [(1.0, 1900.0, []), (2.0, 1500.0, ["sw_power_cap"]), (3.0, 1950.0, []), (4.0, 1960.0, [])]
    cs.max_mhz = 1965.0
    assert cs.window(1.5, 2.5) == {"sm_mhz": 1500.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"]}
    assert cs.window(2.5, 9.0)["sm_mhz"] == 1960.0 and cs.window(2.5, 9.0)["reasons"] == []
    assert cs.window(10.0, 11.0)["sm_mhz"] is None
