"""The one-CTA-per-tile GEMM kernel is the fallback when no CTA pair can be resident; it is selected
with DSN_GEMM_MODE=1cta (read when a context is created), so the parity tests of the linear and
convolution layers are run once more in a child process with that setting."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_linear_and_conv_parity_with_one_cta_kernel():
    env = dict(os.environ, DSN_GEMM_MODE="1cta")
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_linear.py"), os.path.join(ROOT, "tests", "test_gpu_conv_layer.py")]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout
