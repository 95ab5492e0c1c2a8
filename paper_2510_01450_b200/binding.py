"""ctypes binding of ``liblla.so``: the same names as ``include/lla.h``, argument marshalling only.

Every function takes device tensors (anything with ``data_ptr()``; torch is used by callers for
memory and streams only) or raw integer addresses, and returns nothing; a non-zero status from the
library raises ``LlaError``.  There is no CPU fallback: if the shared library is missing the first
call raises, telling how to build it.
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path

_PKG = Path(__file__).resolve().parent
# LLA_LIBRARY selects another build of the same library (the bounds-checking debug build, liblla_debug.so)
_LIB_PATH = Path(os.environ["LLA_LIBRARY"]) if os.environ.get("LLA_LIBRARY") else _PKG / "liblla.so"
_lib = None

LLA_BF16, LLA_F32 = 0, 1
LLA_IMPL_AUTO, LLA_IMPL_SIMT, LLA_IMPL_TENSOR = 0, 1, 2
LLA_STATUS_WORDS = 8
LLA_PHASE_ALL, LLA_PHASE_DIRECT, LLA_PHASE_ITERATIVE = 0, 1, 2
STATUS_ROWS_AT_CAP, STATUS_BAD_PIVOT, STATUS_TIMEOUT, STATUS_ITER_SUM, STATUS_BOUNDS, STATUS_BOUNDS_SITE = 0, 1, 2, 3, 4, 5
LLA_RIDGE_DEFINITION, LLA_RIDGE_PRINTED = 0, 1
LLA_CG_PRECISE_ALL, LLA_CG_PRECISE_NONE = -1, -2
LLA_DEBUG_NO_LOADS = 1

EXPORTS = (
    "lla_forward", "lla_forward_f32", "lla_decode", "lla_decode_f32", "lla_forward_ex", "lla_decode_ex",
    "lla_forward_host", "lla_decode_host", "lla_decode_noalloc", "lla_forward_workspace_bytes", "lla_decode_workspace_bytes",
    "lla_decode_default_splits", "lla_status_string", "lla_version", "lla_backward_ex", "lla_backward_workspace_bytes",
)


class BackwardParams(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
        ("dout", ctypes.c_void_p), ("rho", ctypes.c_void_p), ("stats", ctypes.c_void_p),
        ("dq", ctypes.c_void_p), ("dk", ctypes.c_void_p), ("dv", ctypes.c_void_p),
        ("B", ctypes.c_int), ("H", ctypes.c_int), ("n", ctypes.c_int), ("d", ctypes.c_int),
        ("out_dtype", ctypes.c_int), ("dout_dtype", ctypes.c_int),
        ("scale", ctypes.c_float), ("lambda_", ctypes.c_float),
        ("max_iters", ctypes.c_int), ("tol", ctypes.c_float), ("head_rows", ctypes.c_int),
        ("device_status", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p), ("iters", ctypes.c_void_p), ("dlambda", ctypes.c_void_p), ("impl", ctypes.c_int), ("kv_heads", ctypes.c_int),
        ("window", ctypes.c_int), ("cg_precondition", ctypes.c_int),
        ("block_mask", ctypes.c_void_p), ("block_mask_stride", ctypes.c_longlong), ("q_rows", ctypes.c_int),
        ("debug_wait_clocks", ctypes.c_longlong), ("debug_flags", ctypes.c_int),
    ]


class LlaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class ForwardParams(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
        ("B", ctypes.c_int), ("H", ctypes.c_int), ("n", ctypes.c_int), ("d", ctypes.c_int), ("dv", ctypes.c_int),
        ("in_dtype", ctypes.c_int), ("out_dtype", ctypes.c_int),
        ("scale", ctypes.c_float), ("lambda_", ctypes.c_float),
        ("causal", ctypes.c_int), ("max_iters", ctypes.c_int), ("tol", ctypes.c_float),
        ("head_rows", ctypes.c_int), ("impl", ctypes.c_int), ("phases", ctypes.c_int),
        ("rho", ctypes.c_void_p), ("stats", ctypes.c_void_p), ("iters", ctypes.c_void_p),
        ("device_status", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p), ("lambda_rows", ctypes.c_void_p), ("ridge_mode", ctypes.c_int),
        ("q_rows", ctypes.c_int), ("kv_heads", ctypes.c_int), ("window", ctypes.c_int),
        ("cg_precise_iters", ctypes.c_int),
        ("q_strides", ctypes.c_longlong * 3), ("k_strides", ctypes.c_longlong * 3), ("v_strides", ctypes.c_longlong * 3),
        ("out_strides", ctypes.c_longlong * 3), ("block_mask", ctypes.c_void_p), ("block_mask_stride", ctypes.c_longlong),
        ("cg_precondition", ctypes.c_int), ("debug_wait_clocks", ctypes.c_longlong),
        ("debug_flags", ctypes.c_int),
    ]


class DecodeParams(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("kcache", ctypes.c_void_p), ("vcache", ctypes.c_void_p),
        ("lens", ctypes.c_void_p), ("out", ctypes.c_void_p),
        ("B", ctypes.c_int), ("H", ctypes.c_int), ("Lmax", ctypes.c_int), ("d", ctypes.c_int), ("dv", ctypes.c_int),
        ("in_dtype", ctypes.c_int), ("out_dtype", ctypes.c_int),
        ("scale", ctypes.c_float), ("lambda_", ctypes.c_float),
        ("splits", ctypes.c_int), ("impl", ctypes.c_int),
        ("device_status", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p), ("lambda_units", ctypes.c_void_p), ("ridge_mode", ctypes.c_int),
        ("kv_heads", ctypes.c_int), ("block_table", ctypes.c_void_p), ("page_size", ctypes.c_int),
        ("max_pages", ctypes.c_int), ("num_pages", ctypes.c_int), ("window", ctypes.c_int),
        ("debug_wait_clocks", ctypes.c_longlong), ("debug_flags", ctypes.c_int),
    ]


def load():
    """Load ``liblla.so`` and declare the prototypes.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2510_01450_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    fwd = [vp, vp, vp, vp, i, i, i, i, i, f, f, i, vp]
    dec = [vp, vp, vp, vp, vp, i, i, i, i, i, f, f, vp]
    lib.lla_forward.argtypes = fwd
    lib.lla_forward_f32.argtypes = fwd
    lib.lla_decode.argtypes = dec
    lib.lla_decode_f32.argtypes = dec
    lib.lla_forward_host.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, f, f, i, vp]
    lib.lla_decode_host.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, f, vp]
    lib.lla_decode_noalloc.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, f, i, vp]
    lib.lla_decode_noalloc.restype = i
    lib.lla_forward_ex.argtypes = [ctypes.POINTER(ForwardParams)]
    lib.lla_decode_ex.argtypes = [ctypes.POINTER(DecodeParams)]
    lib.lla_backward_ex.argtypes = [ctypes.POINTER(BackwardParams)]
    lib.lla_backward_ex.restype = i
    lib.lla_backward_workspace_bytes.argtypes = [i, i, i, i]
    lib.lla_backward_workspace_bytes.restype = sz
    for name in ("lla_forward", "lla_forward_f32", "lla_decode", "lla_decode_f32", "lla_forward_ex",
                 "lla_decode_ex", "lla_forward_host", "lla_decode_host", "lla_decode_noalloc", "lla_version",
                 "lla_decode_default_splits"):
        getattr(lib, name).restype = i
    lib.lla_decode_default_splits.argtypes = [i, i, i]
    lib.lla_forward_workspace_bytes.argtypes = [i, i, i, i, i, i, i]
    lib.lla_forward_workspace_bytes.restype = sz
    lib.lla_decode_workspace_bytes.argtypes = [i, i, i, i, i, i, i]
    lib.lla_decode_workspace_bytes.restype = sz
    lib.lla_status_string.argtypes = [i]
    lib.lla_status_string.restype = ctypes.c_char_p
    lib.lla_version.argtypes = []
    _lib = lib
    return lib


def _p(x):
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return ctypes.c_void_p(x.data_ptr())
    return ctypes.c_void_p(int(x))


def _check(rc: int, where: str):
    if rc != 0:
        raise LlaError(rc, where)


def status_string(status: int) -> str:
    return load().lla_status_string(int(status)).decode()


def lla_version() -> int:
    return int(load().lla_version())


def lla_forward(q, k, v, out, B, H, n, d, dv, scale, lam, causal=1, stream=0):
    _check(load().lla_forward(_p(q), _p(k), _p(v), _p(out), B, H, n, d, dv, scale, lam, int(causal), _p(stream)),
           "lla_forward")


def lla_forward_f32(q, k, v, out, B, H, n, d, dv, scale, lam, causal=1, stream=0):
    _check(load().lla_forward_f32(_p(q), _p(k), _p(v), _p(out), B, H, n, d, dv, scale, lam, int(causal),
                                  _p(stream)), "lla_forward_f32")


def lla_decode(q, kcache, vcache, lens, out, B, H, Lmax, d, dv, scale, lam, stream=0):
    _check(load().lla_decode(_p(q), _p(kcache), _p(vcache), _p(lens), _p(out), B, H, Lmax, d, dv, scale, lam,
                             _p(stream)), "lla_decode")


def lla_decode_f32(q, kcache, vcache, lens, out, B, H, Lmax, d, dv, scale, lam, stream=0):
    _check(load().lla_decode_f32(_p(q), _p(kcache), _p(vcache), _p(lens), _p(out), B, H, Lmax, d, dv, scale, lam,
                                 _p(stream)), "lla_decode_f32")


def lla_forward_host(q, k, v, out, B, H, n, d, dv, in_dtype, out_dtype, scale, lam, causal=1, stream=0):
    """Host-buffer form: q, k, v, out are host tensors/addresses; synchronises ``stream``."""
    _check(load().lla_forward_host(_p(q), _p(k), _p(v), _p(out), B, H, n, d, dv, in_dtype, out_dtype, scale, lam,
                                   int(causal), _p(stream)), "lla_forward_host")


def lla_decode_host(q, kcache, vcache, lens, out, B, H, Lmax, d, dv, in_dtype, out_dtype, scale, lam, stream=0):
    _check(load().lla_decode_host(_p(q), _p(kcache), _p(vcache), _p(lens), _p(out), B, H, Lmax, d, dv, in_dtype,
                                  out_dtype, scale, lam, _p(stream)), "lla_decode_host")


def lla_forward_ex(q, k, v, out, B, H, n, d, dv, scale, lam, causal=1, in_dtype=LLA_BF16, out_dtype=LLA_BF16,
                   max_iters=0, tol=0.0, head_rows=0, impl=LLA_IMPL_AUTO, phases=0, rho=None, stats=None, iters=None,
                   device_status=None, workspace=None, workspace_bytes=0, stream=0, lambda_rows=None,
                   ridge_mode=LLA_RIDGE_DEFINITION, q_rows=0, kv_heads=0, window=0, cg_precise_iters=0,
                   debug_wait_clocks=0, debug_flags=0, cg_precondition=0, q_strides=None, k_strides=None, v_strides=None,
                   out_strides=None, block_mask=None, block_mask_stride=0):
    p = ForwardParams()
    p.block_mask, p.block_mask_stride = _p(block_mask), block_mask_stride
    for name, val in (("q_strides", q_strides), ("k_strides", k_strides), ("v_strides", v_strides), ("out_strides", out_strides)):
        if val is not None:
            setattr(p, name, (ctypes.c_longlong * 3)(*[int(x) for x in val]))
    p.cg_precondition = cg_precondition
    p.debug_wait_clocks, p.debug_flags = debug_wait_clocks, debug_flags
    p.kv_heads, p.window, p.cg_precise_iters = kv_heads, window, cg_precise_iters
    p.q, p.k, p.v, p.out = _p(q), _p(k), _p(v), _p(out)
    p.B, p.H, p.n, p.d, p.dv = B, H, n, d, dv
    p.in_dtype, p.out_dtype = in_dtype, out_dtype
    p.scale, p.lambda_, p.causal = scale, lam, int(causal)
    p.max_iters, p.tol, p.head_rows, p.impl, p.phases = max_iters, tol, head_rows, impl, phases
    p.rho, p.stats, p.iters, p.device_status = _p(rho), _p(stats), _p(iters), _p(device_status)
    p.workspace, p.workspace_bytes, p.stream = _p(workspace), workspace_bytes, _p(stream)
    p.lambda_rows, p.ridge_mode, p.q_rows = _p(lambda_rows), ridge_mode, q_rows
    _check(load().lla_forward_ex(ctypes.byref(p)), "lla_forward_ex")


def lla_decode_ex(q, kcache, vcache, lens, out, B, H, Lmax, d, dv, scale, lam, in_dtype=LLA_BF16,
                  out_dtype=LLA_BF16, splits=0, impl=LLA_IMPL_AUTO, device_status=None, workspace=None,
                  workspace_bytes=0, stream=0, lambda_units=None, ridge_mode=LLA_RIDGE_DEFINITION, kv_heads=0, block_table=None,
                  page_size=0, max_pages=0, num_pages=0, window=0, debug_wait_clocks=0, debug_flags=0):
    p = DecodeParams()
    p.window = window
    p.debug_wait_clocks, p.debug_flags = debug_wait_clocks, debug_flags
    p.kv_heads = kv_heads
    p.block_table, p.page_size, p.max_pages, p.num_pages = _p(block_table), page_size, max_pages, num_pages
    p.q, p.kcache, p.vcache, p.lens, p.out = _p(q), _p(kcache), _p(vcache), _p(lens), _p(out)
    p.B, p.H, p.Lmax, p.d, p.dv = B, H, Lmax, d, dv
    p.in_dtype, p.out_dtype = in_dtype, out_dtype
    p.scale, p.lambda_, p.splits, p.impl = scale, lam, splits, impl
    p.device_status, p.workspace, p.workspace_bytes, p.stream = _p(device_status), _p(workspace), workspace_bytes, _p(stream)
    p.lambda_units, p.ridge_mode = _p(lambda_units), ridge_mode
    _check(load().lla_decode_ex(ctypes.byref(p)), "lla_decode_ex")


def lla_backward_ex(q, k, v, out, dout, rho, stats, dq, dk, dv, B, H, n, d, scale, lam, out_dtype=LLA_F32,
                    dout_dtype=LLA_F32, max_iters=0, tol=0.0, head_rows=0, device_status=None, workspace=None,
                    workspace_bytes=0, stream=0, impl=LLA_IMPL_AUTO, iters=None, dlambda=None, kv_heads=0, window=0,
                    cg_precondition=0, block_mask=None, block_mask_stride=0, q_rows=0, debug_wait_clocks=0, debug_flags=0):
    p = BackwardParams()
    p.q_rows = q_rows
    p.debug_wait_clocks, p.debug_flags = debug_wait_clocks, debug_flags
    p.kv_heads, p.window, p.cg_precondition = kv_heads, window, cg_precondition
    p.block_mask, p.block_mask_stride = _p(block_mask), block_mask_stride
    p.impl, p.iters, p.dlambda = impl, _p(iters), _p(dlambda)
    p.q, p.k, p.v, p.out, p.dout = _p(q), _p(k), _p(v), _p(out), _p(dout)
    p.rho, p.stats, p.dq, p.dk, p.dv = _p(rho), _p(stats), _p(dq), _p(dk), _p(dv)
    p.B, p.H, p.n, p.d = B, H, n, d
    p.out_dtype, p.dout_dtype = out_dtype, dout_dtype
    p.scale, p.lambda_ = scale, lam
    p.max_iters, p.tol, p.head_rows = max_iters, tol, head_rows
    p.device_status, p.workspace, p.workspace_bytes, p.stream = _p(device_status), _p(workspace), workspace_bytes, _p(stream)
    _check(load().lla_backward_ex(ctypes.byref(p)), "lla_backward_ex")


def lla_backward_workspace_bytes(B, H, n, d) -> int:
    return int(load().lla_backward_workspace_bytes(B, H, n, d))


NOALLOC_SCRATCH_BYTES = 64 << 20


def lla_decode_noalloc(q, kcache, vcache, lens, out, B, H, Lmax, d, dv, scale, lam, in_dtype=LLA_BF16,
                       out_dtype=LLA_BF16, splits=0, stream=0):
    """Split-key decode for callers that may not allocate device memory (a pre-planned serving loop,
    a host framework that forbids cudaMalloc after start-up): the partial moments live in a fixed
    64 MiB array inside the library instead of a workspace.  Raises LlaError(status 3) when
    B*H*splits records do not fit.  Calls that may overlap on the GPU race on that array."""
    _check(load().lla_decode_noalloc(_p(q), _p(kcache), _p(vcache), _p(lens), _p(out), B, H, Lmax, d, dv,
                                     in_dtype, out_dtype, scale, lam, splits, _p(stream)), "lla_decode_noalloc")


def lla_forward_workspace_bytes(B, H, n, d, dv, in_dtype=LLA_BF16, impl=LLA_IMPL_AUTO) -> int:
    return int(load().lla_forward_workspace_bytes(B, H, n, d, dv, in_dtype, impl))


def lla_decode_workspace_bytes(B, H, Lmax, d, dv, in_dtype=LLA_BF16, splits=1) -> int:
    return int(load().lla_decode_workspace_bytes(B, H, Lmax, d, dv, in_dtype, splits))


def lla_decode_default_splits(B, H, Lmax) -> int:
    return int(load().lla_decode_default_splits(B, H, Lmax))
