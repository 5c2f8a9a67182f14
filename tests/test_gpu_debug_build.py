"""The bounds-checked build (-DEP_DEBUG): every index the kernels compute for themselves is tested before use and a
wrong one would raise a status instead of faulting.  A child process loads that build and runs the smoke pass of the
whole hot path against the oracle; its status word must stay clean."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_smoke_pass_on_the_bounds_checked_build():
    from paper_2604_01000_b200 import build as cuda_build
    lib = cuda_build.build(debug=True)
    assert os.path.exists(lib)
    env = dict(os.environ, EP_USE_DEBUG_LIBRARY="1")
    code = ("import __graft_entry__ as g, paper_2604_01000_b200.binding as b; "
            "assert b.library_path().endswith('libembedpart_debug.so'); g.smoke()")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "smoke ok" in r.stdout, (r.stdout[-1500:], r.stderr[-3000:])
