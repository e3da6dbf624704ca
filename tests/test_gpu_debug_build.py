"""The debug build of the library (host-side assertions, `python -m paper_2407_19775_b200.build --debug`) on a GPU: same bits,
overlapping buffers refused.  The binding loads one library per process, so the case runs as a child with BQ_LIB set."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_debug_build_same_bits_and_overlaps_refused():
    from paper_2407_19775_b200 import build
    lib = build.build_debug()
    env = dict(os.environ, BQ_LIB=lib)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_build_case.py")], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "debug build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
