"""bench.py --gpus N outside a torchrun environment starts the N ranks itself (no GPU needed:
the function that would run the command is replaced)."""
import os
import sys
import types

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench


def _args(gpus):
    return types.SimpleNamespace(gpus=gpus)


def test_single_gpu_runs_in_this_process(monkeypatch):
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    called = []
    assert bench.maybe_relaunch(_args(1), ["--steps", "5"], run=called.append) is None
    assert called == []


def test_a_rank_of_a_running_job_does_not_relaunch(monkeypatch):
    monkeypatch.setenv("WORLD_SIZE", "4")
    called = []
    assert bench.maybe_relaunch(_args(4), ["--gpus", "4"], run=called.append) is None
    assert called == []


def test_gpus_n_starts_n_local_ranks(monkeypatch):
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    seen = []

    def fake_run(cmd):
        seen.append(cmd)
        return 7

    argv = ["--gpus", "8", "--steps", "20", "--warmup", "5"]
    assert bench.maybe_relaunch(_args(8), argv, run=fake_run) == 7
    (cmd,) = seen
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and "--nproc-per-node=8" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    port = int(cmd[cmd.index("--master-port") + 1])
    assert 1024 <= port <= 65535
    script = cmd.index(os.path.join(ROOT, "bench.py"))
    assert cmd[script + 1:] == argv           # the ranks get the caller's flags, --gpus included


def test_launcher_command_is_what_the_scaling_runs_use():
    cmd = bench.launcher_command(2, ["--gpus", "2"], 29511)
    assert cmd == [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                   "--master-addr", "127.0.0.1", "--master-port", "29511",
                   os.path.join(ROOT, "bench.py"), "--gpus", "2"]
