"""The bounds-checking build of the library (libfc_debug.so: the same kernels compiled with -DFC_DEBUG_BOUNDS, every
computed store guarded, a violated guard sets FC_DEV_BAD_INDEX and skips the store) run through the small parity cases.
It stands in for a memory checker: the cases pass, and none of them sees the status bit."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_parity_cases_pass_on_the_bounds_checking_build():
    env = dict(os.environ, FC_LIB="debug")
    pick = "tiny or ragged or edge or small or outputs_stay or select_bit_exact or ignores_rows or shapes or compact_tiny"
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-q", "-x",
                        "-m", "gpu", "-k", pick, "-p", "no:cacheprovider"],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
