"""`bench.py --gpus N` starts N ranks: the launch command, the relaunch decision, and a real two-rank start on
CPU (gloo) through that command."""
import json
import os
import subprocess
import sys

from paper_2605_16154_b200 import launch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_relaunch_only_without_a_launcher_environment():
    assert not launch.needs_relaunch(1, {})
    assert launch.needs_relaunch(2, {})
    assert launch.needs_relaunch(8, {"PATH": "/bin"})
    assert not launch.needs_relaunch(2, {"WORLD_SIZE": "2", "RANK": "0"})
    assert not launch.needs_relaunch(2, {"RANK": "1"})


def test_launch_command_for_two_ranks():
    cmd = launch.torchrun_command(2, "/x/bench.py", ["--gpus", "2", "--steps", "4"], port=12345)
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "12345"
    assert cmd[-5:] == ["/x/bench.py", "--gpus", "2", "--steps", "4"]
    assert 1024 < launch.free_port() < 65536


def test_two_ranks_start_and_rank_zero_reports_both():
    cmd = launch.torchrun_command(2, os.path.join(ROOT, "tests", "launch_probe.py"), [])
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert lines == [{"n_gpus": 2, "slowest": 1.0}]


def test_run_length_defaults():
    assert launch.default_steps("C1") == 10 and launch.default_steps("C4") == 50
    assert launch.default_steps("C4", "reference") == 3
