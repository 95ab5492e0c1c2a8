"""The bounds-checking debug build (python -m paper_2510_01450_b200.build --debug-bounds): the same sources compiled
with -DLLA_DEBUG_BOUNDS, whose kernels check the index of their global stores against the extent that the launch
geometry implies and count violations in the status words instead of trapping.  (The GPU pool offers no memory
checker, so this is the stand-in: small shapes, every kernel family, status words read back.)"""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

from paper_2510_01450_b200 import binding as L

ROOT = Path(__file__).resolve().parent.parent
DEBUG_LIB = ROOT / "paper_2510_01450_b200" / "liblla_debug.so"


@pytest.mark.gpu
def test_debug_build_finds_no_store_out_of_range():
    assert DEBUG_LIB.exists(), "build it with: python -m paper_2510_01450_b200.build --debug-bounds"
    env = dict(os.environ, LLA_LIBRARY=str(DEBUG_LIB))
    res = subprocess.run([sys.executable, str(ROOT / "tests" / "debug_bounds_run.py")], env=env, capture_output=True,
                         text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    report = json.loads(res.stdout.strip().splitlines()[-1])
    assert report["library"] == str(DEBUG_LIB)
    assert len(report["cases"]) == 8
    for case in report["cases"]:
        st = case["status"]
        assert st[L.STATUS_BOUNDS] == 0 and st[L.STATUS_BOUNDS_SITE] == 0, case
        assert st[L.STATUS_TIMEOUT] == 0 and st[L.STATUS_BAD_PIVOT] == 0, case
        assert case["err"] <= (1e-5 if "fp32" in case["name"] else 2e-3), case


def test_debug_library_exports_the_same_entry_points():
    if not DEBUG_LIB.exists():
        pytest.skip("debug library not built")
    import ctypes
    lib = ctypes.CDLL(str(DEBUG_LIB))
    for name in ("lla_forward", "lla_forward_ex", "lla_forward_host", "lla_decode", "lla_decode_ex", "lla_decode_noalloc",
                 "lla_backward_ex", "lla_forward_workspace_bytes", "lla_backward_workspace_bytes", "lla_version"):
        assert hasattr(lib, name), name
