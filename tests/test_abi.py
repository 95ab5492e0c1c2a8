"""Host-only checks of the C ABI: the library loads, exports every symbol the header declares, and
rejects bad arguments before touching a device."""
import ctypes
import os
import re
from pathlib import Path

import pytest

from paper_2510_01450_b200 import binding, build

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_functions():
    text = (ROOT / "include" / "lla.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lla_[a-z0-9_]+)\s*\(", text)))


def test_exports_match_header(lib):
    declared = _declared_functions()
    assert set(declared) == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings(lib):
    assert binding.lla_version() >= 100
    assert binding.status_string(0) == "ok"
    for code in range(1, 6):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert binding.status_string(99) == "unknown status"


def test_struct_layouts_match_c(tmp_path):
    # every field offset and the size of the three parameter structs: the ctypes mirrors against what a C
    # compiler makes of include/lla.h
    import subprocess
    structs = (("lla_forward_params", binding.ForwardParams), ("lla_decode_params", binding.DecodeParams),
               ("lla_backward_params", binding.BackwardParams))
    lines = []
    for cname, cls in structs:
        lines.append(f'  printf("%zu", sizeof({cname}));\n')
        for f, _ in cls._fields_:
            lines.append(f'  printf(" %zu", offsetof({cname}, {"lambda" if f == "lambda_" else f}));\n')
        lines.append('  printf("\\n");\n')
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "lla.h"\nint main(void) {\n' + "".join(lines)
                   + "  return 0; }\n")
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", str(ROOT / "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.strip().splitlines()
    for (cname, cls), line in zip(structs, out):
        got = [int(x) for x in line.split()]
        assert got == [ctypes.sizeof(cls)] + [getattr(cls, f).offset for f, _ in cls._fields_], cname


def test_argument_validation_without_device(lib):
    ok_ptr = 0x1000
    args = dict(B=1, H=1, n=8, d=64, dv=64, scale=0.125, lam=1e-3)

    def fwd(**kw):
        a = {**args, **kw}
        q = kw.get("q", ok_ptr)
        return lib.lla_forward(q, ok_ptr, ok_ptr, ok_ptr, a["B"], a["H"], a["n"], a["d"], a["dv"],
                               a["scale"], a["lam"], 1, None)

    assert fwd(q=None) == 1
    assert fwd(n=0) == 1
    assert fwd(lam=-1.0) == 1
    assert fwd(scale=float("nan")) == 1
    assert fwd(q=0x1004) == 1            # misaligned
    assert fwd(d=32, dv=32) == 2
    assert fwd(d=64, dv=16) == 2
    assert lib.lla_decode(ok_ptr, ok_ptr, ok_ptr, None, ok_ptr, 1, 1, 8, 64, 64, 0.125, 1e-3, None) == 1
    assert lib.lla_decode(ok_ptr, ok_ptr, ok_ptr, ok_ptr, ok_ptr, 1, 1, 0, 64, 64, 0.125, 1e-3, None) == 1
    assert lib.lla_decode(ok_ptr, ok_ptr, ok_ptr, ok_ptr, ok_ptr, 1, 1, 8, 48, 48, 0.125, 1e-3, None) == 2
    assert lib.lla_forward_ex(None) == 1
    p = binding.DecodeParams()
    p.q = p.kcache = p.vcache = p.lens = p.out = ok_ptr
    p.B, p.H, p.Lmax, p.d, p.dv, p.scale, p.lambda_ = 1, 1, 4096, 64, 64, 0.125, 1e-3
    p.splits = 4                          # explicit split without workspace
    assert lib.lla_decode_ex(ctypes.byref(p)) == 3
    with pytest.raises(binding.LlaError):
        binding.lla_forward(None, ok_ptr, ok_ptr, ok_ptr, 1, 1, 8, 64, 64, 0.125, 1e-3)


def test_validation_of_the_position_options(lib):
    # grouped heads, windows, paged caches and the backward's arguments are checked before any device call
    ok = 0x1000

    def fwd(**kw):
        p = binding.ForwardParams()
        p.q = p.k = p.v = p.out = ok
        p.B, p.H, p.n, p.d, p.dv, p.scale, p.lambda_, p.causal = 1, 4, 512, 64, 64, 0.125, 1e-3, 1
        p.in_dtype = p.out_dtype = binding.LLA_BF16
        for name, val in kw.items():
            setattr(p, name, val)
        return lib.lla_forward_ex(ctypes.byref(p))

    assert fwd(kv_heads=3) == 1                    # H is not a multiple
    assert fwd(kv_heads=-1) == 1
    assert fwd(window=-5) == 1
    assert fwd(window=200, causal=0) == 2          # a window needs the causal order
    assert fwd(window=50) == 2                     # below the direct-row threshold (96)
    assert fwd(q_rows=600) == 1                    # more queries than keys
    L3 = ctypes.c_longlong * 3
    assert fwd(q_strides=L3(512 * 64, 64, 4 * 64 + 4)) == 1     # a row stride that is not a multiple of 8 elements
    assert fwd(out_strides=L3(512 * 64, -64, 64)) == 1
    assert fwd(cg_precondition=2) == 1
    assert fwd(debug_flags=8) == 1

    def dec(**kw):
        p = binding.DecodeParams()
        p.q = p.kcache = p.vcache = p.lens = p.out = ok
        p.B, p.H, p.Lmax, p.d, p.dv, p.scale, p.lambda_ = 2, 4, 1024, 64, 64, 0.125, 1e-3
        p.in_dtype = p.out_dtype = binding.LLA_BF16
        p.splits = 1
        for name, val in kw.items():
            setattr(p, name, val)
        return lib.lla_decode_ex(ctypes.byref(p))

    assert dec(kv_heads=3) == 1
    assert dec(block_table=ok, page_size=96, max_pages=16, num_pages=64) == 1      # not a multiple of 128
    assert dec(block_table=ok, page_size=128, max_pages=4, num_pages=64) == 1      # 4 pages cannot hold Lmax keys
    assert dec(block_table=ok, page_size=128, max_pages=8, num_pages=64, window=256) == 1
    assert dec(window=-1) == 1

    def bwd(**kw):
        p = binding.BackwardParams()
        for f in ("q", "k", "v", "out", "dout", "rho", "stats", "dq", "dk", "dv"):
            setattr(p, f, ok)
        p.B, p.H, p.n, p.d, p.scale, p.lambda_ = 1, 4, 256, 64, 0.125, 1e-3
        p.out_dtype = p.dout_dtype = binding.LLA_F32
        p.workspace, p.workspace_bytes = 0x10000, 1 << 40
        for name, val in kw.items():
            setattr(p, name, val)
        return lib.lla_backward_ex(ctypes.byref(p))

    assert bwd(dq=None) == 1
    assert bwd(d=16) == 2
    assert bwd(workspace_bytes=1024) == 3
    assert bwd(workspace=0x10010) == 3             # not 256-byte aligned
    assert bwd(kv_heads=3) == 1
    assert bwd(impl=7) == 1
    # the pass's own fp32 vectors and row records (8 + 4 floats a row), six bf16 operand arrays (y, -t and the upstream gradient as hi + lo
    # pairs), then the scratch of the forward's CG kernel that it runs: fp16 copy of k + a status word, Gram sums and
    # preconditioner matrices per block of 128 keys (2 blocks, 4 heads)
    assert binding.lla_backward_workspace_bytes(1, 4, 256, 64) == (4 * 4 * 256 * (4 * 64 + 8 + 4) + 6 * 4 * 256 * 64 * 2
                                                                  + 4 * 256 * 64 * 2 + 256
                                                                  + 4 * 2 * (64 * 64 + 64) * 4 + 4 * 2 * 64 * 64 * 2)


def test_workspace_and_split_arithmetic(lib):
    # tensor-core forward: fp16 copy of k + a status word (d = 128 adds per-SM slots, which need the device's SM count)
    assert binding.lla_forward_workspace_bytes(4, 8, 1024, 64, 64) == (4 * 8 * 1024 * 64 * 2 + 256          # fp16 copy of k, status word
                                                                       + 32 * 8 * (64 * 64 + 64) * 4     # Gram sums, 8 blocks of 128 keys
                                                                       + 32 * 8 * 64 * 64 * 2)           # preconditioner matrices
    assert binding.lla_forward_workspace_bytes(1, 1, 256, 16, 16, in_dtype=binding.LLA_F32) == 0
    # unsplit: optional record buffer for the two-kernel tensor-core path (bf16, d = 64), else none
    assert binding.lla_decode_workspace_bytes(2, 4, 4096, 64, 64, splits=1) == 4 * 2 * 4 * (2 * 64 * 64 + 132)
    assert binding.lla_decode_workspace_bytes(2, 4, 4096, 64, 64, in_dtype=binding.LLA_F32, splits=1) == 0
    assert binding.lla_decode_workspace_bytes(2, 4, 4096, 128, 128, splits=1) == 0
    assert binding.lla_decode_workspace_bytes(2, 4, 4096, 64, 64, splits=3) == 4 * 2 * 4 * 3 * (2 * 64 * 64 + 132)
    assert binding.lla_decode_default_splits(64, 16, 8192) == 1          # 1024 blocks already fill the chip
    assert binding.lla_decode_default_splits(1, 16, 8192) == 16          # 512-key floor
    assert binding.lla_decode_default_splits(1, 1, 100) == 1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "liblla.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()
