"""The checked build of the library (-DFAEDKV_DEBUG: device-side bounds checks on computed indices, which record a
failure and skip the access instead of faulting) run over small cases of every call, with 256-byte canaries
around every output.  It stands in for a memory checker, which is not available on the test machines."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_cases_under_the_checked_build():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    sys.path.insert(0, ROOT)
    from paper_2507_20030_b200 import build
    lib = build.build(debug=True)
    env = dict(os.environ, FAEDKV_LIBRARY=lib)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_build_cases.py")], env=env, capture_output=True,
                       text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "cases ok" in r.stdout


def test_canary_helper_catches_a_write_past_the_end():
    """The guard helper itself: a byte written behind (or before) the tensor is reported."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from helpers import Guarded
    g = Guarded((3, 5), torch.float32, 0.0)
    g.check()
    g.raw[Guarded.GUARD + g.nbytes] = 0
    with pytest.raises(AssertionError):
        g.check()
    g = Guarded((4,), torch.bfloat16, 0.0)
    g.raw[Guarded.GUARD - 1] = 1
    with pytest.raises(AssertionError):
        g.check()
