"""The debug build of the library (-DMOSKA_DEBUG_GUARDS): same results, guard words behind every
workspace region.  The GPU part runs in a child process because the binding loads one library
per process (MOSKA_LIB selects it)."""
import ctypes
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libs():
    from paper_2511_06010_b200 import build

    return build.build(), build.build(debug=True)


def test_debug_library_exports_the_same_symbols_and_a_larger_workspace(libs):
    from paper_2511_06010_b200 import binding as M

    regular, debug = (ctypes.CDLL(p) for p in libs)
    for name in M.EXPORTS:
        assert hasattr(debug, name), name
    s = M.shape(64, 32, 8, 128, 512, 512, 8)
    for lib in (regular, debug):
        lib.moska_workspace_bytes.restype = ctypes.c_size_t
    extra = debug.moska_workspace_bytes(ctypes.byref(s)) - regular.moska_workspace_bytes(ctypes.byref(s))
    assert extra == 7 * 256  # bit sets, totals, three work lists, router scores (C > 256), f16 queries
    # the regular build has no guard words to compare
    regular.moska_debug_check_workspace.restype = ctypes.c_int
    rc = regular.moska_debug_check_workspace(None, ctypes.c_size_t(0), ctypes.byref(s), None)
    assert rc == M.ERR_UNSUPPORTED


@pytest.mark.gpu
def test_debug_build_step_parity_and_guard_words(libs):
    env = dict(os.environ, MOSKA_LIB=libs[1])
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_build_case.py")], env=env,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "guard words ok" in r.stdout
