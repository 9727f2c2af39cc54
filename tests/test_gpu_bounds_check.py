"""The checked build of the library (-DDNNS_BOUNDS_CHECK): the rebuild kernels compare every data-dependent
index (keep lists, source elements, mask bits) with its extent, count violations and redirect the access
instead of faulting.  A second process loads that build, runs the path on small models against the oracle
and reports the count, which must be zero.  (compute-sanitizer is not available here; guard words catch stray
writes, this catches stray reads.)"""
import os
import subprocess
import sys

import pytest

from paper_2309_06973_b200 import build as build_mod

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_no_index_leaves_its_extent():
    lib = build_mod.build(checked=True)
    env = dict(os.environ, DNNS_LIBRARY=lib)
    out = subprocess.run([sys.executable, os.path.join(HERE, "bounds_check_run.py")], env=env, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-2000:]
    assert out.stdout.strip().splitlines()[-1] == "violations 0", out.stdout[-500:]
