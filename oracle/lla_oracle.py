"""ctypes loader for the float64 CPU oracle (``lla_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
bench's CPU-baseline leg.  The CUDA library never imports this module and this
module never imports the CUDA package.

The arithmetic lives in the C file (paper Section 2.3, Eq. "query_specific" and
Eq. "lla", evaluated by explicit moments and a dense Cholesky solve); this
module only builds the shared object with gcc, marshals numpy arrays and picks
rows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "lla_oracle.c"
_LIB = _HERE / "liblla_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile ``lla_oracle.c`` into ``liblla_oracle.so`` next to it (gcc, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        vp, i32, f64, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_longlong
        lib.lla_oracle_forward_rows.restype = i32
        lib.lla_oracle_forward_rows.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, f64, f64,
                                                i32, vp, i64, vp, vp, vp, vp]
        lib.lla_oracle_decode.restype = i32
        lib.lla_oracle_decode.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, f64, f64,
                                          vp, vp]
        lib.lla_oracle_forward_rows_ex.restype = i32
        lib.lla_oracle_forward_rows_ex.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, f64, f64,
                                                   vp, i32, i32, vp, i64, vp, vp, vp, vp]
        lib.lla_oracle_decode_ex.restype = i32
        lib.lla_oracle_decode_ex.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, f64, f64,
                                             vp, i32, vp, vp]
        lib.lla_oracle_threads.restype = i32
        lib.lla_oracle_threads.argtypes = []
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle's loops will use."""
    return int(_load().lla_oracle_threads())


def _as_input(*arrays):
    """Return contiguous arrays of one common dtype (float32 or float64) and the in_f32 flag."""
    arrays = [np.asarray(a) for a in arrays]
    if all(a.dtype == np.float32 for a in arrays):
        return [np.ascontiguousarray(a) for a in arrays], 1
    return [np.ascontiguousarray(a, dtype=np.float64) for a in arrays], 0


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


RIDGE_MODES = {"definition": 0, "printed": 1}


def _ridge(lam, count):
    """Scalar ridge and optional per-row array (float64, ``count`` entries)."""
    if np.ndim(lam) == 0:
        return float(lam), None
    arr = np.ascontiguousarray(np.asarray(lam, dtype=np.float64).reshape(-1))
    assert arr.size == count, (arr.size, count)
    return 0.0, arr


def forward_rows(q, k, v, scale, lam, causal=True, rows=None, want_aux=False, ridge_mode="definition"):
    """LLA outputs for selected query rows.

    ``lam`` is a scalar or one ridge per query row ``[B,H,n]`` (per-token regularisation).
    ``ridge_mode``: "definition" (raw weights, ridge lambda: Eq. "query_specific") or "printed"
    (Algorithm 1/2 as printed: lambda added in the max-subtracted frame).
    q, k: [B,H,n,d]; v: [B,H,n,dv]; float32 (holds bf16 exactly) or float64.
    rows: 1-D int64 array of flat row indices ``(b*H + h)*n + i`` (default: every row).
    Returns ``out [n_rows, dv]`` float64, and with ``want_aux`` also
    ``rho [n_rows, d]``, ``aux [n_rows, 3] = (m, omega, delta)`` and ``status [n_rows]``.
    """
    (q, k, v), in_f32 = _as_input(q, k, v)
    B, H, n, d = q.shape
    dv = v.shape[-1]
    assert k.shape == (B, H, n, d) and v.shape == (B, H, n, dv)
    if rows is None:
        rows = np.arange(B * H * n, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    assert rows.ndim == 1 and (rows.size == 0 or (rows.min() >= 0 and rows.max() < B * H * n))
    out = np.empty((rows.size, dv), dtype=np.float64)
    rho = np.empty((rows.size, d), dtype=np.float64) if want_aux else None
    aux = np.empty((rows.size, 3), dtype=np.float64) if want_aux else None
    status = np.zeros(rows.size, dtype=np.int32)
    lam0, lam_rows = _ridge(lam, B * H * n)
    rc = _load().lla_oracle_forward_rows_ex(_ptr(q), _ptr(k), _ptr(v), in_f32, B, H, n, d, dv,
                                            float(scale), lam0, _ptr(lam_rows), RIDGE_MODES[ridge_mode],
                                            int(bool(causal)), _ptr(rows), rows.size, _ptr(out), _ptr(rho),
                                            _ptr(aux), _ptr(status))
    if rc < 0:
        raise MemoryError("oracle work buffer allocation failed")
    if want_aux:
        return out, rho, aux, status
    return out


def forward(q, k, v, scale, lam, causal=True, ridge_mode="definition"):
    """LLA output for every row, shaped [B,H,n,dv] float64."""
    B, H, n, _ = np.asarray(q).shape
    out = forward_rows(q, k, v, scale, lam, causal, ridge_mode=ridge_mode)
    return out.reshape(B, H, n, -1)


def decode(q, kcache, vcache, lens, scale, lam, ridge_mode="definition"):
    """Single-query decode: q [B,H,d], caches [B,H,Lmax,d|dv], lens [B] -> out [B,H,dv] float64.

    ``lam`` is a scalar or one ridge per (sequence, head) ``[B,H]``."""
    (q, kcache, vcache), in_f32 = _as_input(q, kcache, vcache)
    B, H, d = q.shape
    Lmax = kcache.shape[2]
    dv = vcache.shape[-1]
    assert kcache.shape == (B, H, Lmax, d) and vcache.shape == (B, H, Lmax, dv)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    assert lens.shape == (B,) and lens.min() >= 1 and lens.max() <= Lmax
    out = np.empty((B, H, dv), dtype=np.float64)
    status = np.zeros(B * H, dtype=np.int32)
    lam0, lam_units = _ridge(lam, B * H)
    rc = _load().lla_oracle_decode_ex(_ptr(q), _ptr(kcache), _ptr(vcache), in_f32, _ptr(lens), B, H,
                                      Lmax, d, dv, float(scale), lam0, _ptr(lam_units),
                                      RIDGE_MODES[ridge_mode], _ptr(out), _ptr(status))
    if rc < 0:
        raise MemoryError("oracle work buffer allocation failed")
    return out
