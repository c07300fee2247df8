"""Order independence: a case whose kernels sit just below a launch limit (the fused heads kernel at 48 384 bytes
of dynamic shared memory, under the 48 KiB that need no opt-in only without its static part) must also pass as
the first thing a process does, when no earlier test has raised that limit."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_multi_tile_round_alone_in_a_fresh_process():
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu",
                        "tests/test_gpu_learner.py::test_conv_sync_rounds_multi_tile"],
                       cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
