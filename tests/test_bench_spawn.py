"""bench.py starts its own ranks: `--gpus N` without a torchrun environment re-executes the script under
torch.distributed.run with N processes and a rendezvous on 127.0.0.1.  Here the ranks are CPU processes on
gloo and stop after the rendezvous check (one all-reduce), which needs no GPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _clean_env():
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT", "LOCAL_WORLD_SIZE")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    return env


def test_respawn_command_shape():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.respawn_command(["--gpus", "4", "--steps", "2"], 4)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")


def test_two_ranks_start_and_meet():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rendezvous-check"],
                         capture_output=True, text=True, timeout=300, env=_clean_env(), cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    rec = json.loads(lines[0])
    assert rec == {"rendezvous": "ok", "n_gpus": 2, "backend": "gloo"}


def test_one_rank_needs_no_launcher():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1", "--rendezvous-check"],
                         capture_output=True, text=True, timeout=120, env=_clean_env(), cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    assert json.loads(res.stdout.strip().splitlines()[-1])["n_gpus"] == 1
