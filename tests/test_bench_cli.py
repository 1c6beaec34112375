"""bench.py's launcher logic on a machine without a GPU: `--gpus N` with no launcher in the
environment starts N ranks itself, and every rank stops with a plain message when there is no CUDA
device (the product has no CPU path)."""
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_gpus_n_starts_n_ranks_that_refuse_to_run_without_a_device():
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    done = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1",
                           "--warmup", "1"], capture_output=True, text=True, timeout=300, env=env)
    assert done.returncode != 0
    text = done.stdout + done.stderr
    # the launcher stops the other rank as soon as one fails, so only one message is certain
    assert text.count("bench.py needs a CUDA device") >= 1
    assert "ChildFailedError" in text or "local_rank" in text or "FAILED" in text   # it ran under the launcher
