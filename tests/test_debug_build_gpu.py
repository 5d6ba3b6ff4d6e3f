"""The checked build of the library (compiled with -DBB_DEBUG: indices taken from the schedule are tested against
their ranges inside the kernels, a failing test records a status instead of touching memory) runs the small parity
cases of the tensor-core kernel without reporting anything.  It stands in for a memory checker."""
import os
import subprocess
import sys

import pytest

from paper_2007_14062_b200 import build as _build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_cases_pass_under_the_checked_build():
    lib = _build.build(debug=True)
    env = dict(os.environ, BIGBIRD_LIB=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_parity_gpu.py"), "-x", "-q", "-m", "gpu",
                        "-k", "small_cases and fwd or fully_padded and fwd", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
