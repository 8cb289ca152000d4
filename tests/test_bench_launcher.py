"""bench.py starts its own ranks when no launcher did: checked on CPU with gloo ranks (the GPU step replaced
by the row split of the sharded path), and refused cleanly when the devices are not there."""
import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ENV = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}


def test_two_ranks_started_by_the_bench_itself():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=ENV,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["max_over_ranks"] == 2.0
    assert line["row_ranges"] == [[0, 256], [256, 512]]      # two ranks, a full b256 batch each


@pytest.mark.skipif(torch.cuda.is_available() and torch.cuda.device_count() >= 2, reason="two devices are present")
def test_more_ranks_than_devices_is_refused_before_anything_starts():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], env=ENV,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode != 0
    assert "needs 2 CUDA devices" in (r.stderr + r.stdout)
