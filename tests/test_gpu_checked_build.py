"""The checked build of the library (-DUBP_DEBUG, libubp_b200_debug.so): the kernels compare every index they take from
the plan or compute for shared / global memory with its extent and report through the plan's status word instead of
trapping (what stands in for a memory checker here). A process loads one build of the library, so the cases run in a
child process that is pointed at the checked build."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEBUG_LIB = os.path.join(ROOT, "paper_2407_19644_b200", "libubp_b200_debug.so")


def test_checked_build_exports_the_same_symbols():
    import ctypes
    import re
    hdr = open(os.path.join(ROOT, "include", "ubp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(ubp_[a-z0-9_]+)\s*\(", hdr))
    if not os.path.exists(DEBUG_LIB):                          # (a tree that was never built: a minute of nvcc)
        from paper_2407_19644_b200 import build
        build.build(debug=True)
    lib = ctypes.CDLL(DEBUG_LIB)
    assert len(names) > 20
    for name in sorted(names):
        assert hasattr(lib, name), name


@pytest.mark.gpu
def test_checked_build_runs_clean_and_notices_a_damaged_plan():
    if not os.path.exists(DEBUG_LIB):
        from paper_2407_19644_b200 import build
        build.build(debug=True)
    env = dict(os.environ, UBP_B200_LIBRARY=DEBUG_LIB)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "checked_build_cases.py")], env=env, cwd=ROOT,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    assert "checked build ok" in r.stdout and "damaged plan: status" in r.stdout
