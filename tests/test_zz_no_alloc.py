"""Decode through the allocation-free entry point.

Some callers cannot allocate device memory at all: a serving loop whose memory was planned up
front, or a host program that bans cudaMalloc once it is running because a synchronising
allocation stalls every stream.  For them the library keeps the partial-moment records of the
split decode in a fixed array of its own.  This test calls that entry point through the C ABI twice
in a row (the second call reuses the array the first one left dirty, with other data and another
split count) and checks both results against the ordinary entry point given a caller workspace.

Collected last on purpose, so a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2510_01450_b200 import binding as L
from paper_2510_01450_b200 import inputs
from tests.gpu_util import dev, row_err, stream_ptr

pytestmark = pytest.mark.gpu


def _reference(dq, dk, dv_, dl, w, splits):
    nbytes = L.lla_decode_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, splits)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    out = torch.full((w.B, w.H, w.dv), float("nan"), dtype=torch.float32, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, out_dtype=L.LLA_F32,
                    splits=splits, workspace=ws, workspace_bytes=nbytes, stream=stream_ptr())
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_no_alloc_decode_matches_workspace_decode_twice(oracle):
    for seed, splits in ((70, 4), (71, 7)):          # two calls in a row, different data and splits
        w = inputs.CONFIGS[5].shrink(B=3, H=4, n=2048, len_min=1, len_max=2048, seed=seed)
        q, kc, vc, lens = inputs.make_decode(w)
        lens[0] = 2048
        lens[1] = 17                                   # short cache: takes the direct path, no scratch
        dq, dk, dv_ = dev(q, "bf16"), dev(kc, "bf16"), dev(vc, "bf16")
        dl = torch.from_numpy(lens).cuda()
        want = _reference(dq, dk, dv_, dl, w, splits)
        out = torch.full((w.B, w.H, w.dv), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        L.lla_decode_noalloc(dq, dk, dv_, dl, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam,
                             out_dtype=L.LLA_F32, splits=splits, stream=stream_ptr())
        torch.cuda.synchronize()
        if seed != 70:      # (the first call of a process may load the module's kernels)
            assert torch.cuda.mem_get_info()[0] == free_before      # the call took no device memory
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        assert row_err(got, want).max() <= 2e-3       # same tolerance as the parity tests (same kernels: equal)
        ref = oracle.decode(q, kc, vc, lens, w.scale, w.lam)
        assert row_err(got, ref).max() <= 2e-3


def test_no_alloc_default_splits_that_do_not_fit_run_unsplit(oracle):
    # d = 128, 280 (sequence, head) pairs: the default of 2 parts needs 74 MB of records; with splits = 0 the call
    # falls back to one part instead of refusing
    w = inputs.CONFIGS[5].shrink(B=70, H=4, n=1024, d=128, dv=128, len_min=300, len_max=1024, seed=72)
    assert L.lla_decode_default_splits(w.B, w.H, w.n) > 1
    assert L.lla_decode_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16,
                                        L.lla_decode_default_splits(w.B, w.H, w.n)) > L.NOALLOC_SCRATCH_BYTES
    q, kc, vc, lens = inputs.make_decode(w)
    dq, dk, dv_ = dev(q, "bf16"), dev(kc, "bf16"), dev(vc, "bf16")
    dl = torch.from_numpy(lens).cuda()
    out = torch.full((w.B, w.H, w.dv), float("nan"), dtype=torch.float32, device="cuda")
    L.lla_decode_noalloc(dq, dk, dv_, dl, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, out_dtype=L.LLA_F32,
                         splits=0, stream=stream_ptr())
    torch.cuda.synchronize()
    ref = oracle.decode(q, kc, vc, lens, w.scale, w.lam)
    assert row_err(out.cpu().numpy(), ref).max() <= 2e-3


def test_no_alloc_rejects_what_does_not_fit():
    # 64 x 16 (sequence, head) pairs x 8 parts of 33 KB each exceed the 64 MiB array: refused on the host
    ok = 0x1000
    assert L.lla_decode_workspace_bytes(64, 16, 8192, 64, 64, L.LLA_BF16, 8) > L.NOALLOC_SCRATCH_BYTES
    with pytest.raises(L.LlaError) as e:
        L.lla_decode_noalloc(ok, ok, ok, ok, ok, 64, 16, 8192, 64, 64, 0.125, 1e-3, splits=8)
    assert e.value.status == 3
