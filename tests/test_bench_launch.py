"""bench.py's own start of its ranks (no GPU needed): `python bench.py --gpus N` outside a launcher
must re-run itself under torch.distributed.run with N ranks on 127.0.0.1 and keep the NCCL log off
stdout, so that rank 0's one JSON line is all that is printed."""
import importlib.util
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _load_bench():
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_relaunch_builds_the_launcher_command(monkeypatch):
    bench = _load_bench()
    seen = {}

    def fake_call(cmd, env=None):
        seen["cmd"], seen["env"] = cmd, env
        return 0

    monkeypatch.setattr(bench.subprocess, "call", fake_call)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7", "--warmup", "3"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.delenv("NCCL_DEBUG", raising=False)
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert e.value.code == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-6:] == ["--gpus", "4", "--steps", "7", "--warmup", "3"] and cmd[-7].endswith("bench.py")
    assert seen["env"]["NCCL_DEBUG"] == "INFO" and "NCCL_DEBUG_FILE" in seen["env"]


def test_a_launcher_with_the_wrong_rank_count_is_refused(monkeypatch):
    bench = _load_bench()
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4"])
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setenv("RANK", "0")
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert "started 2 ranks" in str(e.value.code)


def test_unknown_workloads_are_refused():
    bench = _load_bench()
    with pytest.raises(SystemExit) as e:
        bench._workload("cfg1_tiny")
    assert "not a bench line" in str(e.value.code)
