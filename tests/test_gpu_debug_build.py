"""The substitutes for a memory checker on a pool where compute-sanitizer is closed: guard bands around
every output and workspace (tests/guard_band_run.py), run against the normal library and against the
checked build (LAGA_DEBUG=1), whose kernels verify every TMA coordinate and global store before making it
and report LAGA_ERR_DEVICE_CHECK instead of a bad access.  Each runs in a process of its own because the
binding picks the library when it is imported."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("debug", ["0", "1"])
def test_guard_bands_stay_intact(debug):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import build
    build.build(debug=(debug == "1"))
    env = dict(os.environ, LAGA_DEBUG=debug)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "guard_band_run.py")], env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-1500:] + out.stderr[-3000:]
    assert "GUARD_BANDS_OK" in out.stdout
