"""GPU parity: the CUDA library, called through its C ABI, against the float64 CPU oracle on the
same seeded inputs.

Gate (written here, as the workloads state it): row-wise relative L2 error
    E_row = max_i |o_i - oracle_i|_2 / |oracle_i|_2
<= 1e-5 for the fp32 path and <= 2e-3 for bf16 inputs with fp32 accumulation.  For bf16 inputs the
gate is taken on an fp32 output buffer: rounding the exact answer to bf16 alone costs up to 2^-8 =
3.9e-3 per element (8 significant bits), so the bf16-output result is additionally checked element by element: within
the rounding of the row's largest binade (half a unit in the last place there) plus half the tolerance times the row's
largest element.
"""
import numpy as np
import pytest
import torch

from paper_2510_01450_b200 import binding as L
from paper_2510_01450_b200 import inputs
from tests.gpu_util import LLA_DT, dev, elem_err, forward, row_err, stream_ptr

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5
TOL_BF16 = 2e-3


def _check_bf16_output(got_bf16, ref):
    ref2 = ref.reshape(-1, ref.shape[-1])
    got2 = got_bf16.reshape(-1, ref.shape[-1])
    top = np.abs(ref2).max(axis=1, keepdims=True)
    half_ulp = 2.0 ** (np.floor(np.log2(top)) - 8)          # rounding to bf16 (8 significant bits) in the top binade
    assert (np.abs(got2 - ref2) <= half_ulp + 0.5 * TOL_BF16 * top).all()


def test_config1_fp32_full(oracle):
    w = inputs.CONFIGS[1]
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    dq, dk, dv_ = dev(q, "f32"), dev(k, "f32"), dev(v, "f32")
    out = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.float32, device="cuda")
    L.lla_forward_f32(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, 1, stream_ptr())
    torch.cuda.synchronize()
    err = row_err(out.cpu().numpy(), ref)
    assert err.max() <= TOL_F32, err.max()


@pytest.mark.parametrize("impl", [L.LLA_IMPL_SIMT, L.LLA_IMPL_AUTO])
def test_config2_bf16_full(oracle, impl):
    w = inputs.CONFIGS[2]
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    got = forward(w, q, k, v, out_dtype="f32", impl=impl, device_status=status)
    err = row_err(got, ref)
    assert err.max() <= TOL_BF16, err.max()
    assert elem_err(got, ref).max() <= TOL_BF16
    st = status.cpu().numpy()
    assert st[L.STATUS_ROWS_AT_CAP] == 0 and st[L.STATUS_BAD_PIVOT] == 0 and st[L.STATUS_TIMEOUT] == 0
    # the plain entry point (bf16 output)
    dq, dk, dv_ = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    out = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.bfloat16, device="cuda")
    L.lla_forward(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, 1, stream_ptr())
    torch.cuda.synchronize()
    _check_bf16_output(out.float().cpu().numpy().astype(np.float64), ref)


def test_config3_regression_reduced_full_rows(oracle):
    w = inputs.CONFIGS[3].shrink(B=1, H=2, n=1300)       # two segment boundaries, ragged tail
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    err = row_err(forward(w, q, k, v, out_dtype="f32"), ref)
    assert err.max() <= TOL_BF16, err.max()


def test_config3_full_size_sampled_rows(oracle):
    w = inputs.CONFIGS[3]
    q, k, v = inputs.make_prefill(w)
    rows = inputs.sample_rows(w, per_head=96, heads=3, dense_below=4 * w.d)
    ref = oracle.forward_rows(q, k, v, w.scale, w.lam, rows=rows)
    got = forward(w, q, k, v, out_dtype="f32").reshape(-1, w.dv)[rows]
    err = row_err(got, ref)
    assert err.max() <= TOL_BF16, err.max()


@pytest.mark.parametrize("impl", [L.LLA_IMPL_SIMT, L.LLA_IMPL_TENSOR])
def test_config4_reduced_full_rows(oracle, impl):
    w = inputs.CONFIGS[4].shrink(H=2, n=1100)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    err = row_err(forward(w, q, k, v, out_dtype="f32", impl=impl, device_status=status), ref)
    assert err.max() <= TOL_BF16, err.max()
    st = status.cpu().tolist()
    assert st[L.STATUS_ROWS_AT_CAP] == 0 and st[L.STATUS_BAD_PIVOT] == 0 and st[L.STATUS_TIMEOUT] == 0


def test_config4_full_size_sampled_rows(oracle):
    w = inputs.CONFIGS[4]
    q, k, v = inputs.make_prefill(w)
    rows = inputs.sample_rows(w, per_head=48, heads=2, dense_below=2 * w.d + 16)
    ref = oracle.forward_rows(q, k, v, w.scale, w.lam, rows=rows)
    got = forward(w, q, k, v, out_dtype="f32").reshape(-1, w.dv)[rows]
    err = row_err(got, ref)
    assert err.max() <= TOL_BF16, err.max()


def test_config5_decode_full(oracle):
    w = inputs.CONFIGS[5]
    q, kc, vc, lens = inputs.make_decode(w)
    ref = oracle.decode(q, kc, vc, lens, w.scale, w.lam)
    dq, dk, dv_ = dev(q, "bf16"), dev(kc, "bf16"), dev(vc, "bf16")
    dl = torch.from_numpy(lens).cuda()
    out32 = torch.empty((w.B, w.H, w.dv), dtype=torch.float32, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out32, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam,
                    out_dtype=L.LLA_F32, stream=stream_ptr())
    out16 = torch.empty((w.B, w.H, w.dv), dtype=torch.bfloat16, device="cuda")
    L.lla_decode(dq, dk, dv_, dl, out16, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, stream_ptr())
    torch.cuda.synchronize()
    err = row_err(out32.cpu().numpy(), ref)
    assert err.max() <= TOL_BF16, err.max()
    _check_bf16_output(out16.float().cpu().numpy().astype(np.float64), ref)


@pytest.mark.parametrize("dtype,d", [("bf16", 64), ("f32", 16), ("bf16", 16), ("bf16", 128), ("f32", 64)])
def test_decode_matches_oracle_and_splits_agree(oracle, dtype, d):
    w = inputs.CONFIGS[5].shrink(B=3, H=2, n=1500, d=d, dv=d, dtype=dtype, len_min=1, len_max=1500, seed=50 + d)
    q, kc, vc, lens = inputs.make_decode(w)
    lens[0], lens[1] = 1, 1500                 # one cached pair; a full cache
    ref = oracle.decode(q, kc, vc, lens, w.scale, w.lam)
    dq, dk, dv_ = dev(q, dtype), dev(kc, dtype), dev(vc, dtype)
    dl = torch.from_numpy(lens).cuda()
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for splits in (1, 3, 8):
        nbytes = L.lla_decode_workspace_bytes(w.B, w.H, w.n, d, d, LLA_DT[dtype], splits)
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        out = torch.full((w.B, w.H, d), float("nan"), dtype=torch.float32, device="cuda")
        L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                        out_dtype=L.LLA_F32, splits=splits, workspace=ws, workspace_bytes=nbytes,
                        stream=stream_ptr())
        torch.cuda.synchronize()
        err = row_err(out.cpu().numpy(), ref)
        assert err.max() <= tol, (splits, err.max())
    # unsplit and without the optional record buffer (the streaming kernel then solves in its epilogue)
    out1 = torch.full((w.B, w.H, d), float("nan"), dtype=torch.float32, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out1, w.B, w.H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                    out_dtype=L.LLA_F32, splits=1, stream=stream_ptr())
    torch.cuda.synchronize()
    assert row_err(out1.cpu().numpy(), ref).max() <= tol
    # decode of the last token equals the last prefill row on the same data
    np.testing.assert_allclose(out.cpu().numpy()[0], vc[0, :, 0], rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("impl", [L.LLA_IMPL_SIMT, L.LLA_IMPL_AUTO])
def test_decode_unused_slots_and_late_maximum(oracle, impl):
    """Slots past lens[b] may hold anything (here NaN) and must not leak into the result; and a cache
    whose first 64 keys score ~70 units (2^101) below the rest forces the tensor path to give up its first
    pass, whose weights are relative to the first tile's maximum, and stream the cache again with the true maximum."""
    w = inputs.CONFIGS[5].shrink(B=2, H=2, n=1200, len_min=300, len_max=1200, seed=61)
    q, kc, vc, lens = inputs.make_decode(w)
    lens[:] = [1111, 333]
    qn = q / (np.linalg.norm(q, axis=-1, keepdims=True) ** 2)           # q.qn = 1
    kc[:, :, :64] += (-70.0 / w.scale) * qn[:, :, None, :]             # scaled score of the first tile ~ -70
    kc = inputs.round_to_bf16(kc)
    ref = oracle.decode(q, kc, vc, lens, w.scale, w.lam)
    for b in range(w.B):
        kc[b, :, lens[b]:] = np.nan
        vc[b, :, lens[b]:] = np.nan
    dq, dk, dv_ = dev(q, "bf16"), dev(kc, "bf16"), dev(vc, "bf16")
    dl = torch.from_numpy(lens).cuda()
    for splits in (1, 2):
        nbytes = L.lla_decode_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, splits)
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
        out = torch.full((w.B, w.H, w.dv), float("nan"), dtype=torch.float32, device="cuda")
        L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, out_dtype=L.LLA_F32,
                        splits=splits, impl=impl, device_status=status, workspace=ws, workspace_bytes=nbytes,
                        stream=stream_ptr())
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.isfinite(got).all(), splits
        assert row_err(got, ref).max() <= TOL_BF16, (splits, row_err(got, ref).max())
        assert status.cpu().numpy()[L.STATUS_TIMEOUT] == 0


@pytest.mark.parametrize("n", [1, 2, 31, 127, 128, 129, 300])
def test_ragged_and_tiny_lengths(oracle, n):
    w = inputs.CONFIGS[2].shrink(B=2, H=1, n=n, seed=100 + n)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    err = row_err(forward(w, q, k, v, out_dtype="f32"), ref)
    assert err.max() <= TOL_BF16, err.max()


@pytest.mark.parametrize("dtype,d,n", [("f32", 16, 200), ("bf16", 16, 200), ("f32", 64, 400), ("f32", 128, 300)])
def test_other_shapes_and_dtypes(oracle, dtype, d, n):
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=n, d=d, dv=d, dtype=dtype, seed=7 + d)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    err = row_err(forward(w, q, k, v, out_dtype="f32"), ref)
    assert err.max() <= (TOL_F32 if dtype == "f32" else TOL_BF16), err.max()


def test_noncausal(oracle):
    for n in (40, 333):                                   # below and above the direct-solve threshold
        w = inputs.CONFIGS[2].shrink(B=1, H=2, n=n, seed=11)
        q, k, v = inputs.make_prefill(w)
        ref = oracle.forward(q, k, v, w.scale, w.lam, causal=False)
        err = row_err(forward(w, q, k, v, out_dtype="f32", causal=False), ref)
        assert err.max() <= TOL_BF16, (n, err.max())


def test_large_scores_and_ridge_rescale(oracle):
    # scale 8x the usual: row maxima of several units, so the ridge lambda*exp(-m) matters
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=512, seed=12)
    q, k, v = inputs.make_prefill(w)
    scale = 8.0 * w.scale
    ref = oracle.forward(q, k, v, scale, w.lam)
    dq, dk, dv_ = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    out = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.dv, scale, w.lam, out_dtype=L.LLA_F32,
                     max_iters=96, stream=stream_ptr())
    torch.cuda.synchronize()
    err = row_err(out.cpu().numpy(), ref)
    assert err.max() <= TOL_BF16, err.max()


def test_softmax_limit_on_device():
    # lambda -> infinity: the output tends to softmax attention (Eq. "local_constant")
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=384, lam=1e7, seed=13)
    q, k, v = inputs.make_prefill(w)
    got = forward(w, q, k, v, out_dtype="f32")
    tq, tk, tv = (torch.from_numpy(x).double() for x in (q, k, v))
    s = (tq @ tk.transpose(-1, -2)) * w.scale
    s = s.masked_fill(~torch.tril(torch.ones(w.n, w.n, dtype=torch.bool)), float("-inf"))
    ref = (torch.softmax(s, dim=-1) @ tv).numpy()
    assert row_err(got, ref).max() <= 1e-4


def test_saved_tensors_match_oracle(oracle):
    # rho and (m, omega, delta) as Algorithm 1 stores them for the backward pass
    w = inputs.CONFIGS[2].shrink(B=1, H=1, n=400, seed=14)
    q, k, v = inputs.make_prefill(w)
    ref, rho_ref, aux_ref, _ = oracle.forward_rows(q, k, v, w.scale, w.lam, want_aux=True)
    rho = torch.zeros((1, 1, w.n, w.d), dtype=torch.float32, device="cuda")
    stats = torch.zeros((1, 1, w.n, 3), dtype=torch.float32, device="cuda")
    iters = torch.zeros((1, 1, w.n), dtype=torch.int32, device="cuda")
    got = forward(w, q, k, v, out_dtype="f32", rho=rho, stats=stats, iters=iters)
    assert row_err(got, ref).max() <= TOL_BF16
    assert row_err(rho.cpu().numpy(), rho_ref).max() <= 2e-3
    # (m, omega, delta): m is the shift the kernel formed its weights with -- the row maximum in the oracle and in the
    # direct rows, any convenient value elsewhere (Eq. "lla" does not depend on it) -- and omega, delta are sums of
    # the weights exp(score - m); what is fixed is m + log omega and m + log delta
    st = stats.cpu().numpy().reshape(-1, 3).astype(np.float64)
    np.testing.assert_allclose(st[:, 0] + np.log(st[:, 1]), aux_ref[:, 0] + np.log(aux_ref[:, 1]), rtol=0, atol=2e-3)
    np.testing.assert_allclose(st[:, 0] + np.log(st[:, 2]), aux_ref[:, 0] + np.log(aux_ref[:, 2]), rtol=0, atol=2e-3)
    direct_rows = w.d + w.d // 2 - 1
    np.testing.assert_allclose(st[:direct_rows], aux_ref[:direct_rows], rtol=2e-3, atol=1e-6)
    it = iters.cpu().numpy().ravel()
    direct = w.d + w.d // 2 - 1            # bf16 inputs: rows seeing fewer than 1.5 d keys are solved directly
    assert (it[:direct] == -1).all() and (it[direct:] > 0).all()


def test_head_rows_disabled_still_converges_for_late_rows(oracle):
    # with the direct path off, CG handles every row; late rows must still meet the gate
    w = inputs.CONFIGS[2].shrink(B=1, H=1, n=512, seed=15)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    got = forward(w, q, k, v, out_dtype="f32", head_rows=-1, max_iters=64)
    err = row_err(got, ref)
    assert err[4 * w.d:].max() <= TOL_BF16


def test_host_buffer_entry_points(oracle):
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=300, seed=16)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    hq, hk, hv = (torch.from_numpy(x).to(torch.bfloat16).pin_memory() for x in (q, k, v))
    hout = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.float32).pin_memory()
    for _ in range(2):
        L.lla_forward_host(hq, hk, hv, hout, w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, L.LLA_F32, w.scale, w.lam, 1,
                           stream_ptr())
        assert row_err(hout.numpy(), ref).max() <= TOL_BF16
    # enough (batch, head) units and bytes for the chunked form (upload, kernels and download of the
    # chunks overlap on separate streams); pageable output buffer on purpose
    w = inputs.CONFIGS[2].shrink(B=3, H=3, n=640, seed=18)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    hq, hk, hv = (torch.from_numpy(x).to(torch.bfloat16).pin_memory() for x in (q, k, v))
    hout = torch.full((w.B, w.H, w.n, w.dv), float("nan"), dtype=torch.float32)
    L.lla_forward_host(hq, hk, hv, hout, w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, L.LLA_F32, w.scale, w.lam, 1, stream_ptr())
    assert row_err(hout.numpy(), ref).max() <= TOL_BF16
    wd = inputs.CONFIGS[5].shrink(B=3, H=2, n=700, len_min=5, len_max=700, seed=17)
    dq, kc, vc, lens = inputs.make_decode(wd)
    dref = oracle.decode(dq, kc, vc, lens, wd.scale, wd.lam)
    hq, hk, hv = (torch.from_numpy(x).to(torch.bfloat16).pin_memory() for x in (dq, kc, vc))
    hl = torch.from_numpy(lens)
    hout = torch.empty((wd.B, wd.H, wd.dv), dtype=torch.float32).pin_memory()
    L.lla_decode_host(hq, hk, hv, hl, hout, wd.B, wd.H, wd.n, wd.d, wd.dv, L.LLA_BF16, L.LLA_F32, wd.scale,
                      wd.lam, stream_ptr())
    assert row_err(hout.numpy(), dref).max() <= TOL_BF16


def test_bounded_waits_run_out_and_the_context_stays_usable(oracle):
    # Failure detection without a fault: with the kernel's copy-issuing warp told to issue nothing, no barrier of a
    # block is ever completed, so every role's bounded wait runs out (cap 2^20 clocks, about half a millisecond)
    # with no copy or MMA in flight; the blocks release their tensor memory and leave, the call reports the
    # time-outs in the status words, and the next call on the same context is correct.
    w = inputs.CONFIGS[2].shrink(B=1, H=1, n=256, seed=41)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    got = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR, device_status=status,
                  debug_wait_clocks=1 << 20, debug_flags=L.LLA_DEBUG_NO_LOADS)
    tiles = 2                                            # rows 95..127 of the first tile, the second tile
    assert status.cpu().tolist()[L.STATUS_TIMEOUT] == tiles
    assert np.isnan(got[0, 0, 95:]).all()                # the iterative rows were left unwritten
    assert row_err(got[0, 0, :95], ref[0, 0, :95]).max() <= TOL_BF16     # the direct rows (fewer than 96 keys) are another kernel
    for _ in range(2):
        got = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR, device_status=status)
        assert status.cpu().tolist()[L.STATUS_TIMEOUT] == 0
        assert row_err(got, ref).max() <= TOL_BF16


@pytest.mark.parametrize("splits", [1, 3])
def test_decode_bounded_waits_run_out_and_the_context_stays_usable(oracle, splits):
    # the same for the decode's streaming kernel: no copy is issued, every block's waits run out, the blocks leave
    # (their records poisoned, so the solve kernel emits NaN rather than what an earlier call left in the workspace),
    # the time-outs are counted, and the next call is correct
    w = inputs.CONFIGS[5].shrink(B=2, H=2, n=700, len_min=200, len_max=700, seed=340)
    q, kc, vc, lens = inputs.make_decode(w)
    ref = oracle.decode(q, kc, vc, lens, w.scale, w.lam)
    dq, dk, dv_ = dev(q, "bf16"), dev(kc, "bf16"), dev(vc, "bf16")
    dl = torch.from_numpy(lens).cuda()
    nbytes = L.lla_decode_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, splits)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")

    def run(**kw):
        out = torch.full((w.B, w.H, w.dv), 7.0, dtype=torch.float32, device="cuda")
        L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, out_dtype=L.LLA_F32, splits=splits,
                        device_status=status, workspace=ws, workspace_bytes=nbytes, stream=stream_ptr(), **kw)
        torch.cuda.synchronize()
        return out.cpu().numpy(), status.cpu().tolist()

    good, st = run()                                   # leaves valid records of these units in the workspace
    assert st[L.STATUS_TIMEOUT] == 0 and row_err(good, ref).max() <= TOL_BF16
    got, st = run(debug_wait_clocks=1 << 20, debug_flags=L.LLA_DEBUG_NO_LOADS)
    assert w.B * w.H <= st[L.STATUS_TIMEOUT] <= w.B * w.H * splits      # every part that has keys (a short cache's last parts are empty)
    assert np.isnan(got).all()
    got, st = run()
    assert st[L.STATUS_TIMEOUT] == 0 and row_err(got, ref).max() <= TOL_BF16


def test_host_buffer_forward_from_two_threads(oracle):
    # two host threads, each with its own stream and its own problem, in the chunked host-buffer form at the same
    # time: the library's worker streams and events are shared per device, so the calls must not mix them up
    import threading
    jobs = []
    for seed, n in ((31, 640), (32, 512)):
        w = inputs.CONFIGS[2].shrink(B=3, H=3, n=n, seed=seed)
        q, k, v = inputs.make_prefill(w)
        host = tuple(torch.from_numpy(x).to(torch.bfloat16).pin_memory() for x in (q, k, v))
        hout = torch.full((w.B, w.H, w.n, w.dv), float("nan"), dtype=torch.float32).pin_memory()
        jobs.append((w, host, hout, oracle.forward(q, k, v, w.scale, w.lam), torch.cuda.Stream()))
    errors = []

    def work(job):
        w, (hq, hk, hv), hout, _, stream = job
        try:
            for _ in range(6):
                hout.fill_(float("nan"))
                L.lla_forward_host(hq, hk, hv, hout, w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, L.LLA_F32, w.scale, w.lam, 1,
                                   stream.cuda_stream)
                if not np.isfinite(hout.numpy()).all():
                    errors.append("non-finite output")
        except Exception as e:      # noqa: BLE001
            errors.append(repr(e))

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for w, _, hout, ref, _ in jobs:
        assert row_err(hout.numpy(), ref).max() <= TOL_BF16


@pytest.mark.parametrize("dtype,d,n", [("bf16", 64, 700), ("bf16", 128, 400), ("f32", 16, 200)])
def test_ridge_variants_forward(oracle, dtype, d, n):
    # per-token ridge and the ridge of the printed algorithm (both only change lambda'_i)
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=n, d=d, dv=d, dtype=dtype, seed=70 + d)
    q, k, v = inputs.make_prefill(w)
    q = (q * 3.0).astype(np.float32)                      # row maxima well away from 0: the two variants differ
    if dtype == "bf16":
        q = inputs.round_to_bf16(q)
    lam_rows = np.random.default_rng(71).uniform(0.5, 2.0, size=(w.B, w.H, w.n)).astype(np.float32) * w.lam
    dlam = torch.from_numpy(lam_rows).cuda()
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    ref_def = oracle.forward(q, k, v, w.scale, lam_rows.astype(np.float64))
    got = forward(w, q, k, v, out_dtype="f32", lambda_rows=dlam)
    assert row_err(got, ref_def).max() <= tol
    ref_pr = oracle.forward(q, k, v, w.scale, w.lam, ridge_mode="printed")
    got = forward(w, q, k, v, out_dtype="f32", ridge_mode=L.LLA_RIDGE_PRINTED)
    assert row_err(got, ref_pr).max() <= tol
    assert row_err(ref_pr.reshape(-1, d), oracle.forward(q, k, v, w.scale, w.lam).reshape(-1, d)).max() > 10 * tol


@pytest.mark.parametrize("dtype,d", [("bf16", 64), ("f32", 16)])
def test_ridge_variants_decode(oracle, dtype, d):
    w = inputs.CONFIGS[5].shrink(B=3, H=2, n=900, d=d, dv=d, dtype=dtype, len_min=40, len_max=900, seed=72 + d)
    q, kc, vc, lens = inputs.make_decode(w)
    q = (q * 3.0).astype(np.float32)
    if dtype == "bf16":
        q = inputs.round_to_bf16(q)
    lam_units = np.random.default_rng(73).uniform(0.5, 2.0, size=(w.B, w.H)).astype(np.float32) * w.lam
    dq, dk, dv_ = dev(q, dtype), dev(kc, dtype), dev(vc, dtype)
    dl = torch.from_numpy(lens).cuda()
    dlam = torch.from_numpy(lam_units).cuda()
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    for mode, name in ((L.LLA_RIDGE_DEFINITION, "definition"), (L.LLA_RIDGE_PRINTED, "printed")):
        ref = oracle.decode(q, kc, vc, lens, w.scale, lam_units.astype(np.float64), ridge_mode=name)
        out = torch.full((w.B, w.H, d), float("nan"), dtype=torch.float32, device="cuda")
        L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                        out_dtype=L.LLA_F32, splits=1, lambda_units=dlam, ridge_mode=mode, stream=stream_ptr())
        torch.cuda.synchronize()
        assert row_err(out.cpu().numpy(), ref).max() <= tol, name


@pytest.mark.parametrize("d,n", [(64, 1100), (128, 900)])
def test_operand_precision_modes_and_missing_workspace(oracle, d, n):
    # the CG sweeps' on-the-fly operands: bf16 pairs throughout, fp16 from the first iteration, the default mix,
    # and the default without a workspace (no fp16 copy of k: pairs throughout, bit-identical to the first)
    w = inputs.CONFIGS[2 if d == 64 else 4].shrink(B=1, H=2, n=n)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    outs = {}
    for name, kw in (("pairs", dict(cg_precise_iters=L.LLA_CG_PRECISE_ALL)), ("fp16", dict(cg_precise_iters=L.LLA_CG_PRECISE_NONE)),
                     ("three", dict(cg_precise_iters=3)), ("default", {}), ("no_ws", dict(workspace=None, workspace_bytes=0))):
        outs[name] = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR, device_status=status, **kw)
        assert row_err(outs[name], ref).max() <= TOL_BF16, name
        assert elem_err(outs[name], ref).max() <= TOL_BF16, name
        assert status.cpu().tolist()[L.STATUS_TIMEOUT] == 0
    assert np.array_equal(outs["pairs"], outs["no_ws"])      # same arithmetic, same bits
    assert not np.array_equal(outs["pairs"], outs["fp16"])
    # fewer precise iterations cost accuracy, never more than a few 1e-4
    assert row_err(outs["pairs"], ref).max() <= 2.5e-4
    assert row_err(outs["fp16"], ref).max() <= 1.2e-3


@pytest.mark.parametrize("case", ["d64", "d128", "window", "chunk_gqa", "noncausal", "peaked"])
def test_preconditioned_cg_gives_the_same_rows_in_fewer_iterations(oracle, case):
    # cg_precondition = 1: the inverse key covariance per block of 128 keys as preconditioner.  Same solution
    # (it only changes the path of the iteration), fewer iterations where the weights are near uniform, and a
    # row on which the rounded matrix is not positive definite carries on with plain CG.
    kw, okw = {}, {}
    if case == "d64":
        w = inputs.CONFIGS[2].shrink(B=1, H=2, n=1100)
    elif case == "d128":
        w = inputs.CONFIGS[4].shrink(H=2, n=900)
    elif case == "window":
        w = inputs.CONFIGS[2].shrink(B=1, H=2, n=900, seed=91)
        kw = dict(window=300)
    elif case == "chunk_gqa":
        w = inputs.CONFIGS[2].shrink(B=1, H=4, n=800, seed=92)
    elif case == "noncausal":
        w = inputs.CONFIGS[2].shrink(B=1, H=2, n=500, seed=93)
    else:
        w = inputs.CONFIGS[2].shrink(B=1, H=2, n=700, seed=94)
    q, k, v = inputs.make_prefill(w)
    if case == "peaked":
        q = inputs.round_to_bf16(q * np.float32(12.0))       # scores up to +-10: weights far from uniform
    causal = case != "noncausal"
    if case == "window":
        # sampled rows as single queries over exactly their visible keys (the oracle's decode entry point)
        win = kw["window"]
        pos = np.unique(np.concatenate([np.arange(96, 420), np.random.default_rng(5).integers(0, w.n, 150), [w.n - 1]]))
        qs = np.stack([q[0, :, i] for i in pos])
        kc = np.zeros((len(pos), w.H, win, w.d), dtype=np.float32)
        vc = np.zeros((len(pos), w.H, win, w.d), dtype=np.float32)
        cnt = np.zeros(len(pos), dtype=np.int32)
        for s_, i in enumerate(pos):
            lo = max(0, i + 1 - win)
            cnt[s_] = i + 1 - lo
            kc[s_, :, :cnt[s_]] = k[0, :, lo:i + 1]
            vc[s_, :, :cnt[s_]] = v[0, :, lo:i + 1]
        ref = oracle.decode(qs, kc, vc, cnt, w.scale, w.lam).transpose(1, 0, 2).reshape(-1, w.dv)     # [H * rows, dv]
        rows = (np.arange(w.H)[:, None] * w.n + pos[None, :]).reshape(-1)
    elif case == "chunk_gqa":
        rows = None
        kv = 2
        ref = oracle.forward(q, np.repeat(k[:, :kv], w.H // kv, axis=1), np.repeat(v[:, :kv], w.H // kv, axis=1), w.scale, w.lam)
    else:
        rows = None
        ref = oracle.forward(q, k, v, w.scale, w.lam, causal=causal)
    its = {}
    for pc in (0, 1):
        iters = torch.zeros((w.B, w.H, w.n), dtype=torch.int32, device="cuda")
        status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
        if case == "chunk_gqa":
            dq, dk, dv_ = dev(q, "bf16"), dev(np.ascontiguousarray(k[:, :2]), "bf16"), dev(np.ascontiguousarray(v[:, :2]), "bf16")
            out = torch.full((w.B, w.H, w.n, w.dv), float("nan"), dtype=torch.float32, device="cuda")
            nb = L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.dv)
            ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
            L.lla_forward_ex(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, out_dtype=L.LLA_F32, kv_heads=2,
                             cg_precondition=pc, iters=iters, device_status=status, workspace=ws, workspace_bytes=nb,
                             impl=L.LLA_IMPL_TENSOR, stream=stream_ptr())
            torch.cuda.synchronize()
            got = out.cpu().numpy().astype(np.float64)
        else:
            got = forward(w, q, k, v, out_dtype="f32", causal=causal, impl=L.LLA_IMPL_TENSOR, cg_precondition=pc, iters=iters,
                          device_status=status, **kw)
        st = status.cpu().tolist()
        assert st[L.STATUS_TIMEOUT] == 0 and st[L.STATUS_ROWS_AT_CAP] == 0
        cmp = got.reshape(-1, w.dv)[rows] if rows is not None else got
        assert row_err(cmp, ref).max() <= TOL_BF16, (case, pc)
        it = iters.cpu().numpy()
        its[pc] = it[it >= 0].mean()
    if case == "peaked":
        assert its[1] <= 1.5 * its[0]           # no help expected, no harm beyond the restart of failed rows
    else:
        assert its[1] <= 0.75 * its[0], its


@pytest.mark.parametrize("dtype,d,n,impl", [("bf16", 64, 700, L.LLA_IMPL_AUTO), ("bf16", 128, 450, L.LLA_IMPL_AUTO),
                                             ("bf16", 64, 300, L.LLA_IMPL_SIMT), ("f32", 16, 200, L.LLA_IMPL_AUTO)])
def test_strided_layouts_are_read_in_place(oracle, dtype, d, n, impl):
    # tensors kept as [B, n, H, d] (position-major, as many frameworks store them), grouped key/value heads, a padded
    # row pitch for v and an output that is a column slice of a wider buffer: all addressed through the strides
    B, H, Hk = 2, 4, 2
    w = inputs.CONFIGS[2].shrink(B=B, H=H, n=n, d=d, dv=d, dtype=dtype, seed=111 + d)
    q, k, v = inputs.make_prefill(w)
    k, v = k[:, :Hk], v[:, :Hk]
    ref = oracle.forward(q, np.repeat(k, H // Hk, axis=1), np.repeat(v, H // Hk, axis=1), w.scale, w.lam)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    q_bnhd = torch.from_numpy(q).to(tdt).cuda().permute(0, 2, 1, 3).contiguous()            # [B, n, H, d]
    k_bnhd = torch.from_numpy(k).to(tdt).cuda().permute(0, 2, 1, 3).contiguous()            # [B, n, Hk, d]
    pitch = d + 8
    v_pad = torch.zeros((B, Hk, n, pitch), dtype=tdt, device="cuda")                       # rows of d + 8 elements
    v_pad[..., :d] = torch.from_numpy(v).to(tdt).cuda()
    out_wide = torch.full((B, n, H, 2 * d), float("nan"), dtype=torch.float32, device="cuda")   # out in columns d .. 2d
    out_view = out_wide[..., d:]
    nbytes = L.lla_forward_workspace_bytes(B, H, n, d, d, LLA_DT[dtype], impl)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    for pc in ((0, 1) if dtype == "bf16" and impl == L.LLA_IMPL_AUTO else (0,)):
        out_wide.fill_(float("nan"))
        L.lla_forward_ex(q_bnhd, k_bnhd, v_pad, out_view, B, H, n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                         out_dtype=L.LLA_F32, impl=impl, kv_heads=Hk, cg_precondition=pc, workspace=ws if nbytes else None,
                         workspace_bytes=nbytes, stream=stream_ptr(),
                         q_strides=(n * H * d, d, H * d), k_strides=(n * Hk * d, d, Hk * d),
                         v_strides=(Hk * n * pitch, n * pitch, pitch), out_strides=(n * H * 2 * d, 2 * d, H * 2 * d))
        torch.cuda.synchronize()
        got = out_wide[..., d:].permute(0, 2, 1, 3).cpu().numpy()
        assert torch.isnan(out_wide[..., :d]).all()                                          # nothing written beside the slice
        assert row_err(got, ref).max() <= (TOL_F32 if dtype == "f32" else TOL_BF16), pc


@pytest.mark.parametrize("d,n,per_head", [(64, 1500, False), (128, 1100, True)])
def test_block_sparse_forward(oracle, d, n, per_head):
    # a random block mask (about 40 % of the [query tile] x [key block] pairs kept); the blocks of the first head_rows
    # keys and each tile's diagonal blocks are attended whatever the mask says.  The oracle solves sampled rows as
    # single queries over exactly their visible keys (its decode entry point).
    B, H = 1, 3
    w = inputs.CONFIGS[2 if d == 64 else 4].shrink(B=B, H=H, n=n, seed=130 + d)
    q, k, v = inputs.make_prefill(w)
    tiles, blocks = (n + 127) // 128, (n + 63) // 64
    rng = np.random.default_rng(7)
    units = B * H if per_head else 1
    mask = (rng.random((units, tiles, blocks)) < 0.4).astype(np.uint8)
    head_rows = d + d // 2
    dmask = torch.from_numpy(mask).cuda()
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    got = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR, block_mask=dmask,
                  block_mask_stride=tiles * blocks if per_head else 0, device_status=status)
    st = status.cpu().tolist()
    assert st[L.STATUS_TIMEOUT] == 0 and st[L.STATUS_ROWS_AT_CAP] == 0

    def visible(u, i):
        t = i // 128
        keep = np.zeros(i + 1, dtype=bool)
        for c in range(i // 64 + 1):
            on = mask[u if per_head else 0, t, c] != 0 or c * 64 < head_rows or c * 64 + 63 >= t * 128
            if on:
                keep[c * 64:min(i + 1, c * 64 + 64)] = True
        return np.nonzero(keep)[0]

    pos = np.unique(np.concatenate([np.arange(0, 260, 7), rng.integers(0, n, 60), [n - 1]]))
    samples = [(h, i) for h in range(H) for i in pos]
    S = len(samples)
    qs = np.zeros((S, 1, d), dtype=np.float32)
    kc = np.zeros((S, 1, n, d), dtype=np.float32)
    vc = np.zeros((S, 1, n, d), dtype=np.float32)
    cnt = np.zeros(S, dtype=np.int32)
    for s_, (h, i) in enumerate(samples):
        idx = visible(h, i)
        cnt[s_] = len(idx)
        qs[s_, 0] = q[0, h, i]
        kc[s_, 0, :len(idx)] = k[0, h, idx]
        vc[s_, 0, :len(idx)] = v[0, h, idx]
    ref = oracle.decode(qs, kc, vc, cnt, w.scale, w.lam)[:, 0]
    mine = np.stack([got[0, h, i] for h, i in samples])
    assert row_err(mine, ref).max() <= TOL_BF16
    dense = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR)
    assert row_err(np.stack([dense[0, h, n - 1] for h in range(H)]), np.stack([got[0, h, n - 1] for h in range(H)])).max() > 10 * TOL_BF16


def test_values_beyond_the_fp16_range_fall_back_to_pairs(oracle):
    # a key entry of 7e4 cannot be held in fp16: the pre-pass notices and every sweep of the call runs on the bf16
    # inputs.  The entry sits in the last key, which only the last row sees (that row's system is hopelessly
    # ill-conditioned and is left out of the comparison).
    w = inputs.CONFIGS[2].shrink(B=1, H=1, n=600)
    q, k, v = inputs.make_prefill(w)
    k = k.copy()
    k[0, 0, w.n - 1, 3] = inputs.round_to_bf16(np.float32([7.0e4]))[0]
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    got = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR)
    pairs = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR, cg_precise_iters=L.LLA_CG_PRECISE_ALL)
    assert np.array_equal(got[..., :-1, :], pairs[..., :-1, :])
    assert row_err(got[..., :-1, :], ref[..., :-1, :]).max() <= TOL_BF16


def test_forward_d128_with_caller_workspace(oracle):
    # the d = 128 tensor-core kernel keeps its row vectors off chip: in the caller's workspace when one
    # of the advertised size is passed (no allocation inside the call), else in the library's own buffer
    w = inputs.CONFIGS[4].shrink(H=2, n=700)
    q, k, v = inputs.make_prefill(w)
    ref = oracle.forward(q, k, v, w.scale, w.lam)
    nbytes = L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.dv)
    assert nbytes >= 148 * 3 * 128 * 128 * 4
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    got = forward(w, q, k, v, out_dtype="f32", impl=L.LLA_IMPL_TENSOR, workspace=ws, workspace_bytes=nbytes)
    assert row_err(got, ref).max() <= TOL_BF16


@pytest.mark.parametrize("dtype,d,n,nq", [("bf16", 64, 900, 300), ("bf16", 64, 330, 280), ("bf16", 128, 700, 129),
                                           ("f32", 16, 400, 130), ("bf16", 64, 1024, 1)])
def test_chunked_prefill_against_existing_keys(oracle, dtype, d, n, nq):
    # q_rows < n: the last nq positions are the queries (a chunk appended to a cache of n - nq keys).
    # Every such row must equal the same row of the full causal forward.
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=n, d=d, dv=d, dtype=dtype, seed=80 + nq)
    q, k, v = inputs.make_prefill(w)
    off = n - nq
    rows = np.concatenate([np.arange(h * n + off, (h + 1) * n) for h in range(w.B * w.H)]).astype(np.int64)
    ref = oracle.forward_rows(q, k, v, w.scale, w.lam, rows=rows).reshape(w.B, w.H, nq, d)
    dq = dev(np.ascontiguousarray(q[:, :, off:]), dtype)
    dk, dv_ = dev(k, dtype), dev(v, dtype)
    out = torch.full((w.B, w.H, nq, d), float("nan"), dtype=torch.float32, device="cuda")
    iters = torch.zeros((w.B, w.H, nq), dtype=torch.int32, device="cuda")
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    L.lla_forward_ex(dq, dk, dv_, out, w.B, w.H, n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                     out_dtype=L.LLA_F32, q_rows=nq, iters=iters, device_status=status, stream=stream_ptr())
    torch.cuda.synchronize()
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    assert row_err(out.cpu().numpy(), ref).max() <= tol
    st = status.cpu().numpy()
    assert st[L.STATUS_ROWS_AT_CAP] == 0 and st[L.STATUS_BAD_PIVOT] == 0 and st[L.STATUS_TIMEOUT] == 0
    # rows that see fewer keys than the direct-solve threshold are marked -1, the others iterated
    thr = 2 * d if dtype == "f32" else d + d // 2
    seen = off + np.arange(nq) + 1
    it = iters.cpu().numpy()[0, 0]
    assert ((it == -1) == (seen < thr)).all()


@pytest.mark.parametrize("dtype,d,n,H,Hkv", [("bf16", 64, 500, 4, 2), ("bf16", 128, 300, 4, 1), ("f32", 16, 150, 6, 2)])
def test_grouped_kv_heads_forward(oracle, dtype, d, n, H, Hkv):
    # H query heads read H / Hkv-fold shared key/value heads: the oracle sees k, v repeated per query head
    w = inputs.CONFIGS[2].shrink(B=2, H=H, n=n, d=d, dv=d, dtype=dtype, seed=90 + d)
    q, _, _ = inputs.make_prefill(w)
    wk = w.shrink(H=Hkv, seed=91 + d)
    _, k, v = inputs.make_prefill(wk)
    ref = oracle.forward(q, np.repeat(k, H // Hkv, axis=1), np.repeat(v, H // Hkv, axis=1), w.scale, w.lam)
    dq, dk, dv_ = dev(q, dtype), dev(k, dtype), dev(v, dtype)
    out = torch.full((w.B, H, n, d), float("nan"), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq, dk, dv_, out, w.B, H, n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype], out_dtype=L.LLA_F32,
                     kv_heads=Hkv, stream=stream_ptr())
    torch.cuda.synchronize()
    assert row_err(out.cpu().numpy(), ref).max() <= (TOL_F32 if dtype == "f32" else TOL_BF16)
    with pytest.raises(L.LlaError):
        L.lla_forward_ex(dq, dk, dv_, out, w.B, H, n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                         out_dtype=L.LLA_F32, kv_heads=H - 1 if H > 2 else 3, stream=stream_ptr())


@pytest.mark.parametrize("dtype,d,splits", [("bf16", 64, 1), ("bf16", 64, 3), ("f32", 16, 1)])
def test_grouped_kv_heads_decode(oracle, dtype, d, splits):
    H, Hkv = 4, 2
    w = inputs.CONFIGS[5].shrink(B=3, H=H, n=1100, d=d, dv=d, dtype=dtype, len_min=20, len_max=1100, seed=92 + d)
    q, _, _, lens = inputs.make_decode(w)
    _, kc, vc, _ = inputs.make_decode(w.shrink(H=Hkv))
    ref = oracle.decode(q, np.repeat(kc, H // Hkv, axis=1), np.repeat(vc, H // Hkv, axis=1), lens, w.scale, w.lam)
    dq, dk, dv_ = dev(q, dtype), dev(kc, dtype), dev(vc, dtype)
    dl = torch.from_numpy(lens).cuda()
    out = torch.full((w.B, H, d), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = L.lla_decode_workspace_bytes(w.B, H, w.n, d, d, in_dtype=LLA_DT[dtype], splits=splits)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                    out_dtype=L.LLA_F32, splits=splits, workspace=ws, workspace_bytes=nbytes, kv_heads=Hkv,
                    stream=stream_ptr())
    torch.cuda.synchronize()
    assert row_err(out.cpu().numpy(), ref).max() <= (TOL_F32 if dtype == "f32" else TOL_BF16)


def _to_pages(cache, lens, page_size, rng):
    """[B, Hkv, Lmax, d] contiguous cache -> ([num_pages, Hkv, page_size, d] pages in a random order, block table)."""
    B, Hkv, Lmax, d = cache.shape
    max_pages = (Lmax + page_size - 1) // page_size
    need = [(int(l) + page_size - 1) // page_size for l in lens]
    num_pages = sum(need) + 3                       # a few pages nobody owns
    order = rng.permutation(num_pages)
    pages = np.zeros((num_pages, Hkv, page_size, d), dtype=cache.dtype)
    table = np.full((B, max_pages), -1, dtype=np.int32)          # unused entries are never read
    nxt = 0
    for b in range(B):
        for pi in range(need[b]):
            pg = int(order[nxt]); nxt += 1
            lo, hi = pi * page_size, min(Lmax, (pi + 1) * page_size)
            pages[pg, :, : hi - lo] = cache[b, :, lo:hi]
            table[b, pi] = pg
    return pages, table, max_pages, num_pages


@pytest.mark.parametrize("dtype,d,splits,page_size,Hkv", [("bf16", 64, 1, 128, 4), ("bf16", 64, 3, 256, 2),
                                                          ("f32", 16, 1, 128, 4), ("f32", 16, 2, 128, 2)])
def test_paged_cache_decode(oracle, dtype, d, splits, page_size, Hkv):
    H = 4
    w = inputs.CONFIGS[5].shrink(B=4, H=H, n=1200, d=d, dv=d, dtype=dtype, len_min=10, len_max=1200, seed=95 + d)
    q, _, _, lens = inputs.make_decode(w)
    _, kc, vc, _ = inputs.make_decode(w.shrink(H=Hkv))
    ref = oracle.decode(q, np.repeat(kc, H // Hkv, axis=1), np.repeat(vc, H // Hkv, axis=1), lens, w.scale, w.lam)
    rng = np.random.default_rng(96)
    kp, table, max_pages, num_pages = _to_pages(kc, lens, page_size, rng)
    vp, table_v, _, _ = _to_pages(vc, lens, page_size, np.random.default_rng(96))
    assert (table == table_v).all()
    dq, dk, dv_ = dev(q, dtype), dev(kp, dtype), dev(vp, dtype)
    dl, dt = torch.from_numpy(lens).cuda(), torch.from_numpy(table).cuda()
    out = torch.full((w.B, H, d), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = L.lla_decode_workspace_bytes(w.B, H, w.n, d, d, in_dtype=LLA_DT[dtype], splits=splits)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                    out_dtype=L.LLA_F32, splits=splits, workspace=ws, workspace_bytes=nbytes, kv_heads=Hkv,
                    block_table=dt, page_size=page_size, max_pages=max_pages, num_pages=num_pages, stream=stream_ptr())
    torch.cuda.synchronize()
    assert row_err(out.cpu().numpy(), ref).max() <= (TOL_F32 if dtype == "f32" else TOL_BF16)
    with pytest.raises(L.LlaError):
        L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                        out_dtype=L.LLA_F32, block_table=dt, page_size=96, max_pages=max_pages, num_pages=num_pages,
                        stream=stream_ptr())


@pytest.mark.parametrize("dtype,d,splits,window", [("bf16", 64, 1, 300), ("bf16", 64, 2, 1000), ("bf16", 64, 1, 50),
                                                   ("f32", 16, 1, 200), ("f32", 16, 2, 20)])
def test_sliding_window_decode(oracle, dtype, d, splits, window):
    # the query sees the last `window` cached keys: the oracle is given exactly those keys as a cache of its own
    w = inputs.CONFIGS[5].shrink(B=5, H=2, n=1500, d=d, dv=d, dtype=dtype, len_min=10, len_max=1500, seed=97 + d)
    q, kc, vc, lens = inputs.make_decode(w)
    lens[0] = window                      # exactly one window
    lens[1] = window + 1
    kw, vw = np.zeros_like(kc), np.zeros_like(vc)
    cnt = np.minimum(lens, window).astype(np.int32)
    for b in range(w.B):
        kw[b, :, : cnt[b]] = kc[b, :, lens[b] - cnt[b]: lens[b]]
        vw[b, :, : cnt[b]] = vc[b, :, lens[b] - cnt[b]: lens[b]]
    ref = oracle.decode(q, kw, vw, cnt, w.scale, w.lam)
    dq, dk, dv_ = dev(q, dtype), dev(kc, dtype), dev(vc, dtype)
    dl = torch.from_numpy(lens).cuda()
    out = torch.full((w.B, w.H, d), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = L.lla_decode_workspace_bytes(w.B, w.H, w.n, d, d, in_dtype=LLA_DT[dtype], splits=splits)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, d, d, w.scale, w.lam, in_dtype=LLA_DT[dtype],
                    out_dtype=L.LLA_F32, splits=splits, workspace=ws, workspace_bytes=nbytes, window=window,
                    stream=stream_ptr())
    torch.cuda.synchronize()
    assert row_err(out.cpu().numpy(), ref).max() <= (TOL_F32 if dtype == "f32" else TOL_BF16)


@pytest.mark.parametrize("dtype,d,n,window,impl", [("bf16", 64, 900, 200, 0), ("bf16", 64, 900, 96, 0), ("bf16", 64, 700, 333, 1),
                                                   ("bf16", 128, 600, 256, 0), ("f32", 16, 300, 40, 0)])
def test_sliding_window_forward(oracle, dtype, d, n, window, impl):
    # row i sees positions max(0, i + 1 - window) .. i; the oracle solves sampled rows as single queries over
    # exactly those keys (its decode entry point: one "sequence" per sampled row)
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=n, d=d, dv=d, dtype=dtype, seed=98 + d)
    q, k, v = inputs.make_prefill(w)
    got = forward(w, q, k, v, out_dtype="f32", window=window, impl=impl)
    rng = np.random.default_rng(99)
    rows = np.unique(np.concatenate([np.arange(0, min(n, window + 70)), rng.integers(0, n, 120), [n - 1]]))
    S = len(rows)
    qs = np.zeros((S, w.H, d), dtype=np.float32)
    kc = np.zeros((S, w.H, window, d), dtype=np.float32)
    vc = np.zeros((S, w.H, window, d), dtype=np.float32)
    cnt = np.zeros(S, dtype=np.int32)
    for s, i in enumerate(rows):
        lo = max(0, i + 1 - window)
        cnt[s] = i + 1 - lo
        qs[s] = q[0, :, i]
        kc[s, :, : cnt[s]] = k[0, :, lo: i + 1]
        vc[s, :, : cnt[s]] = v[0, :, lo: i + 1]
    ref = oracle.decode(qs, kc, vc, cnt, w.scale, w.lam)                 # [S, H, d]
    err = row_err(got[0][:, rows].transpose(1, 0, 2), ref)
    assert err.max() <= (TOL_F32 if dtype == "f32" else TOL_BF16), (float(err.max()), int(err.argmax()))
    # without the window the late rows differ: the window is really applied
    full = forward(w, q, k, v, out_dtype="f32", impl=impl)
    assert row_err(full[0][:, -1], ref[-1]).max() > 10 * (TOL_F32 if dtype == "f32" else TOL_BF16)


def test_window_with_chunked_queries_and_grouped_heads(oracle):
    # the three position-dependent options together: the last q_rows queries of n keys, a window, shared K/V heads
    d, n, nq, window, H, Hkv = 64, 800, 300, 160, 4, 2
    w = inputs.CONFIGS[2].shrink(B=1, H=H, n=n, d=d, dv=d, seed=110)
    q, _, _ = inputs.make_prefill(w)
    _, k, v = inputs.make_prefill(w.shrink(H=Hkv, seed=111))
    qc = np.ascontiguousarray(q[:, :, n - nq:])
    dq, dk, dv_ = dev(qc, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    out = torch.full((1, H, nq, d), float("nan"), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq, dk, dv_, out, 1, H, n, d, d, w.scale, w.lam, out_dtype=L.LLA_F32, q_rows=nq, kv_heads=Hkv,
                     window=window, stream=stream_ptr())
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    rows = np.unique(np.concatenate([np.arange(0, 40), np.random.default_rng(112).integers(0, nq, 60), [nq - 1]]))
    S = len(rows)
    qs = np.zeros((S, H, d), dtype=np.float32)
    kc = np.zeros((S, H, window, d), dtype=np.float32)
    vc = np.zeros((S, H, window, d), dtype=np.float32)
    kk, vv = np.repeat(k, H // Hkv, axis=1), np.repeat(v, H // Hkv, axis=1)
    for s, r in enumerate(rows):
        pos = n - nq + r
        qs[s] = qc[0, :, r]
        kc[s] = kk[0, :, pos + 1 - window: pos + 1]
        vc[s] = vv[0, :, pos + 1 - window: pos + 1]
    ref = oracle.decode(qs, kc, vc, np.full(S, window, dtype=np.int32), w.scale, w.lam)
    assert row_err(got[0][:, rows].transpose(1, 0, 2), ref).max() <= TOL_BF16
