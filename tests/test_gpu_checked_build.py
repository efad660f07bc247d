"""The checked build of the library (libapms_checked.so, -DAPMS_BOUNDS_CHECK) in place of a memory checker.

In that build every global store of the step's kernels, their streaming loads and the sources of their bulk copies
are validated on the device against the contexts' workspaces and guard regions; an access that would leave its
array is skipped and reported as APMS_ERR_BOUNDS.  Here the guard-byte tests - the edge shapes through every launch
shape, the phase-wise calls, the variants, compared with the oracle - run once more in a child process that loads
the checked library: no accessor may fire, the results must still equal the oracle's, and the self-test that aims
one checked store into guard bytes must see it refused."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_the_ordinary_build_has_no_checked_accessors():
    assert not B.apms_build_is_checked()


def test_guard_and_parity_tests_pass_on_the_checked_build():
    lib = lib_build.build(checked=True)                      # compiled here if it is not there yet
    env = dict(os.environ, APMS_LIBRARY=lib)
    probe = subprocess.run([sys.executable, "-c", "from paper_2008_11343_b200 import binding as B; print(B.apms_build_is_checked())"],
                           capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert probe.stdout.strip() == "True", probe.stdout + probe.stderr        # the child processes do load the checked library
    cmd = [sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_guards.py"), "-m", "gpu", "-x", "-q",
           "-k", "not topk"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=3000, cwd=ROOT, env=env)
    tail = res.stdout[-1500:] + res.stderr[-500:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "skipped" not in res.stdout.splitlines()[-1], tail
