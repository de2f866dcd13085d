"""The multi-GPU plumbing of bench.py on CPU: replicas only, so the only cross-rank step is the
max over ranks of the timings (world size 2, gloo)."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
mine = [10.0 + rank, 5.0 - rank, 1.0]
got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
assert got == [10.0 + world - 1, 5.0, 1.0], got
rate = bench.aggregate_rate(world, 4, got[0])
single = bench.aggregate_rate(1, 4, got[0])
assert abs(rate - world * single) < 1e-9 * rate
dist.barrier()
if rank == 0:
    print("OK", world, flush=True)
dist.destroy_process_group()
"""


def test_max_over_ranks_and_aggregate_rate_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, REPO_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)]
    res = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "OK 2" in res.stdout


def test_single_process_passthrough_and_reference_arm_ranks():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, None) == [1.5, 2.5]
    # 3 linear launches per step, each streaming codes + BF16 scales
    per_step = 3 * (14336 * 4096 // 2 + 14336 * 32 * 2)
    assert bench.weight_bytes() * 3 == per_step
    assert abs(bench.aggregate_rate(2, 10, 1.0) - 2 * 10 * per_step / 1e-3 / 1e9) < 1e-6

    class A:
        steps, warmup, gpus = 1, 0, 2
    assert bench.run_reference(A, rank=1) is None      # ranks other than 0 do no work


def test_gpus_without_a_launcher_starts_the_ranks_or_fails_loudly(monkeypatch):
    # `bench.py --gpus N` with WORLD_SIZE unset re-runs itself under torch.distributed.run with N
    # ranks on 127.0.0.1; with fewer devices than ranks it refuses instead of measuring one GPU
    sys.path.insert(0, ROOT)
    import pytest
    import torch
    import bench
    monkeypatch.setattr(torch.cuda, "device_count", lambda: 1)
    with pytest.raises(SystemExit) as e:
        bench.spawn_ranks(2)
    assert "2" in str(e.value) and "1 CUDA" in str(e.value)
    seen = {}
    monkeypatch.setattr(torch.cuda, "device_count", lambda: 8)
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "20", "--warmup", "5"])
    assert bench.spawn_ranks(4) == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-6:] == ["--gpus", "4", "--steps", "20", "--warmup", "5"] and cmd[-7].endswith("bench.py")
