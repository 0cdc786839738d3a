"""The self-checking build of the library (-DNM_DEBUG_BOUNDS): every address the gathering kernels
(variants 1, 2, 3, 8) derive from index data is range-checked on the device, a violation is recorded in the
handle's status word and the access skipped (no trap).  The small-shape and select-kernel suites run once
more against that build in a child process (the library path is chosen at import time); any recorded
violation surfaces there as NM_ERR_INTERNAL from nm_weights_check and fails the child."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_shapes_under_the_self_checking_build():
    from paper_2507_17301_b200 import build
    lib = build.build(defines=("NM_DEBUG_BOUNDS",), suffix="_debug")
    assert os.path.exists(lib)
    env = dict(os.environ, NM_LIBRARY=lib)
    r = subprocess.run(
        [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
         os.path.join(ROOT, "tests", "test_gpu_conv.py"), os.path.join(ROOT, "tests", "test_gpu_select.py"),
         "-k", "tiny or small_shapes or select_kernel_integer_exact or asymmetric"],
        cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout
