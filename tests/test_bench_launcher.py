"""`bench.py --gpus N` started plainly (no torchrun environment) must start N ranks itself, and both arms must
report the number of ranks that actually ran. Checked on CPU with the script's dry-run mode: gloo ranks that
only sleep, the same launcher, rendezvous, barrier and max-over-ranks protocol as a real run."""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def _run(*argv):
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), *argv], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stdout + p.stderr
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout                       # rank 0 alone prints
    return json.loads(lines[0])


@pytest.mark.parametrize("impl", ["ours", "reference"])
def test_gpus_2_starts_two_ranks(impl):
    line = _run("--gpus", "2", "--steps", "3", "--warmup", "1", "--dry-run", "--impl", impl)
    assert line["n_gpus"] == 2 and line["impl"] == impl
    # rank 1 sleeps twice as long per step as rank 0: the reported time is the slower rank's
    assert line["ms_per_step"] >= 3.9


def test_gpus_1_runs_in_process():
    line = _run("--gpus", "1", "--steps", "2", "--warmup", "1", "--dry-run")
    assert line["n_gpus"] == 1
