"""The checked build of the library (index checks inside the kernels) and a bounded wait running out inside a real
attention kernel: both run in a child process that loads libnsp_checked.so instead of libnsp.so."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent


def test_checked_kernels_match_the_oracle_and_a_withheld_load_times_out_cleanly():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    lib = ROOT / "paper_2609_22755_b200" / "libnsp_checked.so"
    assert lib.exists(), "build it with python -m paper_2609_22755_b200.build"
    env = dict(os.environ, NSP_LIBRARY=str(lib))
    r = subprocess.run([sys.executable, str(ROOT / "tests" / "checked_build_case.py")], env=env, capture_output=True,
                       text=True, timeout=600)
    print(r.stdout)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "fresh plan after the timeout: ok" in r.stdout
