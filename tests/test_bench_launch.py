"""`python bench.py --gpus N` without a launcher starts its own N ranks: the command it builds
gives every rank the environment bench.py reads (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR on
127.0.0.1), and run_ours takes that path before it touches a GPU."""
import json
import os
import subprocess
import sys
import types

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_launch_command_shape():
    import bench
    cmd = bench.rank_launch_command(4, ["--gpus", "4", "--steps", "3"], port=29511)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-5] == os.path.join(ROOT, "bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "3"]


def test_launched_ranks_get_their_environment(tmp_path):
    import bench
    probe = os.path.join(ROOT, "tests", "_rank_env_probe.py")
    cmd = bench.rank_launch_command(2, [str(tmp_path)], script=probe)
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    subprocess.run(cmd, check=True, timeout=300, env=env, stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    assert sorted(g["RANK"] for g in got) == ["0", "1"]
    assert sorted(g["LOCAL_RANK"] for g in got) == ["0", "1"]
    assert all(g["WORLD_SIZE"] == "2" and g["MASTER_ADDR"] == "127.0.0.1" for g in got)
    assert got[0]["MASTER_PORT"] == got[1]["MASTER_PORT"]


def test_gpus_flag_without_launcher_starts_ranks(monkeypatch):
    import bench
    seen = {}
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "1"])
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    with pytest.raises(SystemExit) as e:
        bench.run_ours(types.SimpleNamespace(gpus=2))
    assert e.value.code == 0
    assert seen["cmd"][cmd_index(seen["cmd"], "--nproc-per-node") + 1] == "2"
    assert seen["cmd"][-4:] == ["--gpus", "2", "--steps", "1"]


def cmd_index(cmd, flag):
    return cmd.index(flag)
