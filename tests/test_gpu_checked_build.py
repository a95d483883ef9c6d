"""The checked build (-DEXCP_DEBUG_BOUNDS): every index the kernels form from data is tested before use and a
violation comes back as a status code instead of a fault.  The tool that would normally watch the kernels' memory
accesses is not available where these tests run, so this build stands in for it: the tiny configuration, the
edge sizes, the degenerate value patterns, every code width and every ablation switch run through it in a child
process (its library has a name of its own and never replaces the plain one) and must give the oracle's records
with no check firing."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_suite_under_the_checked_build():
    env = dict(os.environ, EXCP_NVCC_FLAGS="-DEXCP_DEBUG_BOUNDS")
    files = ["tests/test_gpu_parity.py", "tests/test_gpu_bits.py", "tests/test_gpu_ablation.py", "tests/test_gpu_dense.py",
             "tests/test_gpu_w16.py"]
    out = subprocess.run([sys.executable, "-m", "pytest", *files, "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout and "failed" not in out.stdout
