"""bench.py starts its own ranks: `--gpus N` without a launcher's environment re-runs the script under
torch.distributed.run, one rank per GPU. Checked here without a GPU: the command it builds, and that on a machine
without CUDA two ranks really start and a rank stops with a clear message instead of falling back to the CPU."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_launcher_command():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(["--gpus", "4", "--steps", "7"], 4, port=29777)
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29777"
    assert cmd[-5].endswith("bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "7"]


def test_two_ranks_start_and_refuse_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("needs a machine without CUDA")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "1"],
                       capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert r.returncode != 0
    text = r.stdout + r.stderr
    # the launcher ends the other rank as soon as the first one has failed, so only one of the two messages is certain;
    # "of 2" shows that the rank ran inside a two-rank job
    assert "rank 0 of 2: no CUDA device" in text or "rank 1 of 2: no CUDA device" in text, text[-2000:]
