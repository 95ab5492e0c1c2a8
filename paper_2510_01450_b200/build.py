"""Build ``liblla.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Usage: ``python -m paper_2510_01450_b200.build [--force] [--verbose] [--debug-bounds]``

Every ``csrc/*.cu`` is compiled to an object file of its own (in parallel, only when it or a header
is newer than the object) and the objects are linked into one shared library next to the package.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
OBJ = PKG / "build"
LIB = PKG / "liblla.so"
DEBUG_OBJ = OBJ / "debug"
DEBUG_LIB = PKG / "liblla_debug.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(CSRC.glob("*.cu"))


def _headers_mtime() -> float:
    return max(p.stat().st_mtime for p in list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "lla.h"])


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> Path:
    """Compile every ``csrc/*.cu`` and link them into one shared object next to the package.  ``debug_bounds``
    builds ``liblla_debug.so`` instead: the same sources with ``-DLLA_DEBUG_BOUNDS``, whose kernels check the
    indices of their global stores and count violations in the status words (``LLA_LIBRARY`` selects the library
    that the binding loads)."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    hdr = _headers_mtime()
    LIB, OBJ = (DEBUG_LIB, DEBUG_OBJ) if debug_bounds else (globals()["LIB"], globals()["OBJ"])
    if not force and LIB.exists() and LIB.stat().st_mtime >= max([hdr] + [s.stat().st_mtime for s in sources()]):
        return LIB      # up to date (the objects need not exist: only the library travels to a GPU machine)
    OBJ.mkdir(parents=True, exist_ok=True)
    jobs = []
    for src in sources():
        obj = OBJ / (src.stem + ".o")
        if force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, hdr):
            cmd = [nvcc, *NVCC_FLAGS, *(["-DLLA_DEBUG_BOUNDS"] if debug_bounds else []), "-c", "-o", str(obj), str(src)]
            if verbose:
                cmd[1:1] = ["-Xptxas", "-v"]
            jobs.append(cmd)
    if jobs:
        def run(cmd):
            if verbose:
                print(" ".join(cmd), flush=True)
            return subprocess.run(cmd, capture_output=not verbose, text=True)
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as pool:
            for cmd, res in zip(jobs, pool.map(run, jobs)):
                if res.returncode != 0:
                    raise RuntimeError(f"nvcc failed: {' '.join(cmd)}\n{res.stdout or ''}\n{res.stderr or ''}")
    objs = [OBJ / (s.stem + ".o") for s in sources()]
    if jobs or not LIB.exists() or LIB.stat().st_mtime < max(o.stat().st_mtime for o in objs):
        tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run([nvcc, "--shared", "-gencode", "arch=compute_100a,code=sm_100a", "-lcuda", "-o", str(tmp),
                        *map(str, objs)], check=True)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
