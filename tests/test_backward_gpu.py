"""GPU parity of the backward pass: lla_backward_ex, through the C ABI, against the float64 gradient
oracle on the same seeded inputs.

Gate: row-wise relative L2 error of each gradient tensor (one row = one token's dq_i, dk_j or dv_j; see
grad_err for rows whose exact gradient vanishes) <= 2e-3, the forward's bf16-input tolerance: the arithmetic is the same (bf16 inputs, fp32
accumulation, conjugate-gradient solves to a relative residual of 1e-4), with the forward output given
as fp32.  With a bf16 forward output the row term g.o carries that rounding (2^-9 relative), and the
gate for dq and dk is taken relative to the tensor's largest row instead.
"""
import numpy as np
import pytest
import torch

from paper_2510_01450_b200 import binding as L
from paper_2510_01450_b200 import inputs
from tests.gpu_util import LLA_DT, dev, stream_ptr

pytestmark = pytest.mark.gpu

TOL = 2e-3


def grad_err(got, ref):
    """Row-wise |got_i - ref_i| / max(|ref_i|, floor): the gating metric, with a floor of a tenth of the
    median row norm (and 1e-4 absolute) so that rows whose exact gradient is zero or tiny -- the first
    token's dq and dk vanish identically -- are measured against the tensor's scale."""
    d = ref.shape[-1]
    rn = np.linalg.norm(ref.reshape(-1, d), axis=1)
    diff = np.linalg.norm((got - ref).reshape(-1, d), axis=1)
    return diff / np.maximum(rn, max(0.1 * float(np.median(rn)), 1e-4))


def run_backward(w, q, k, v, g, out_dtype="f32", dout_dtype="f32", impl=L.LLA_IMPL_AUTO, window=0, block_mask=None,
                 block_mask_stride=0, **kw):
    dq_, dk_, dv_ = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    dg = dev(g, dout_dtype)
    shape = (w.B, w.H, w.n, w.d)
    out = torch.empty(shape, dtype=torch.float32 if out_dtype == "f32" else torch.bfloat16, device="cuda")
    rho = torch.empty(shape, dtype=torch.float32, device="cuda")
    stats = torch.empty((w.B, w.H, w.n, 3), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq_, dk_, dv_, out, w.B, w.H, w.n, w.d, w.d, w.scale, w.lam, in_dtype=L.LLA_BF16,
                     out_dtype=LLA_DT[out_dtype], rho=rho, stats=stats, stream=stream_ptr(), window=window,
                     block_mask=block_mask, block_mask_stride=block_mask_stride)
    grads = [torch.full(shape, float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    nbytes = L.lla_backward_workspace_bytes(w.B, w.H, w.n, w.d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    L.lla_backward_ex(dq_, dk_, dv_, out, dg, rho, stats, *grads, w.B, w.H, w.n, w.d, w.scale, w.lam,
                      out_dtype=LLA_DT[out_dtype], dout_dtype=LLA_DT[dout_dtype], device_status=status,
                      workspace=ws, workspace_bytes=nbytes, stream=stream_ptr(), impl=impl, window=window,
                      block_mask=block_mask, block_mask_stride=block_mask_stride, **kw)
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert st[L.STATUS_BAD_PIVOT] == 0 and st[L.STATUS_TIMEOUT] == 0
    return [t.cpu().numpy().astype(np.float64) for t in grads]


@pytest.mark.parametrize("d,n,B,H,impl", [(64, 1, 1, 1, 0), (64, 70, 1, 2, 0), (64, 96, 1, 1, 0), (64, 333, 2, 2, 0),
                                          (64, 640, 1, 2, 0), (64, 333, 2, 2, 1), (64, 200, 1, 1, 1),
                                          (128, 150, 1, 1, 0), (128, 420, 1, 2, 0), (128, 420, 1, 2, 1)])
def test_backward_matches_gradient_oracle(backward_oracle, d, n, B, H, impl):
    w = inputs.CONFIGS[2].shrink(B=B, H=H, n=n, d=d, dv=d, seed=200 + n)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    ref = backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    got = run_backward(w, q, k, v, g, impl=impl)
    for name, a, b in zip(("dq", "dk", "dv"), got, ref):
        assert np.isfinite(a).all(), name
        err = grad_err(a, b)
        assert err.max() <= TOL, (name, float(err.max()), int(err.argmax()))


def test_backward_regression_recipe_and_bf16_tensors(backward_oracle):
    # the test-time-regression recipe of Section 4.1 (values linear in the keys, the query is the next key); g and out in bf16
    w = inputs.CONFIGS[3].shrink(B=1, H=2, n=600, seed=231)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w, "bf16")
    ref = backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    got = run_backward(w, q, k, v, g)
    for name, a, b in zip(("dq", "dk", "dv"), got, ref):
        assert grad_err(a, b).max() <= TOL, name
    got16 = run_backward(w, q, k, v, g, out_dtype="bf16", dout_dtype="bf16")
    assert grad_err(got16[2], ref[2]).max() <= TOL
    for a, b in zip(got16[:2], ref[:2]):
        rows = np.linalg.norm(b.reshape(-1, w.d), axis=1)
        diff = np.linalg.norm((a - b).reshape(-1, w.d), axis=1)
        assert diff.max() <= 2.0 ** -8 * rows.max()


def test_backward_bench_shape_one_head(backward_oracle):
    # one head of the bench workload (n = 1024: 16 query tiles by 16 key tiles, the first 95 rows direct)
    w = inputs.CONFIGS[2].shrink(B=1, H=1, seed=260)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    *ref, ref_dlam = backward_oracle.backward(q, k, v, g, w.scale, w.lam, want_dlambda=True)
    iters = torch.full((1, 1, w.n), -1, dtype=torch.int32, device="cuda")
    dlam = torch.full((1, 1, w.n), float("nan"), dtype=torch.float32, device="cuda")
    got = run_backward(w, q, k, v, g, iters=iters, dlambda=dlam)
    for name, a, b in zip(("dq", "dk", "dv"), got, ref):
        err = grad_err(a, b)
        assert err.max() <= TOL, (name, float(err.max()), int(err.argmax()))
    dl = dlam.cpu().numpy().astype(np.float64).ravel()
    assert np.abs(dl - ref_dlam.ravel()).max() <= TOL * np.abs(ref_dlam).max()
    assert np.abs(dl - ref_dlam.ravel())[200:].max() <= TOL * np.abs(ref_dlam.ravel()[200:]).max()
    it = iters.cpu().numpy().ravel()
    assert (it[:95] == -1).all() and (it[95:] > 0).all() and it.max() <= 64


def test_backward_full_bench_workload_sampled_heads(backward_oracle):
    # the whole bench workload (4 x 8 heads, n = 1024) in the launch configuration bench.py times; the oracle
    # checks two of the 32 heads (heads are independent, so it is given those heads' inputs alone)
    w = inputs.CONFIGS[2]
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    got = run_backward(w, q, k, v, g)
    for b, h in ((0, 0), (w.B - 1, w.H - 1)):
        sl = (slice(b, b + 1), slice(h, h + 1))
        ref = backward_oracle.backward(q[sl], k[sl], v[sl], g[sl], w.scale, w.lam)
        for name, a, r in zip(("dq", "dk", "dv"), got, ref):
            err = grad_err(a[sl], r)
            assert err.max() <= TOL, (name, b, h, float(err.max()))


@pytest.mark.parametrize("d,impl", [(64, 0), (128, 0), (64, 1)])
def test_backward_grouped_kv_heads(backward_oracle, d, impl):
    # H query heads over Hkv shared key/value heads: the oracle sees k, v repeated per query head and the
    # shared head's gradient is the sum over its group
    B, H, Hkv, n = 1, 4, 2, 300
    w = inputs.CONFIGS[2].shrink(B=B, H=H, n=n, d=d, dv=d, seed=270 + d)
    q, _, _ = inputs.make_prefill(w)
    _, k, v = inputs.make_prefill(w.shrink(H=Hkv, seed=271 + d))
    g = inputs.make_upstream_grad(w)
    grp = H // Hkv
    rq, rk, rv = backward_oracle.backward(q, np.repeat(k, grp, axis=1), np.repeat(v, grp, axis=1), g, w.scale, w.lam)
    rk = rk.reshape(B, Hkv, grp, n, d).sum(axis=2)
    rv = rv.reshape(B, Hkv, grp, n, d).sum(axis=2)
    dq_, dk_, dv_ = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    dg = dev(g, "f32")
    out = torch.empty((B, H, n, d), dtype=torch.float32, device="cuda")
    rho = torch.empty((B, H, n, d), dtype=torch.float32, device="cuda")
    stats = torch.empty((B, H, n, 3), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq_, dk_, dv_, out, B, H, n, d, d, w.scale, w.lam, out_dtype=L.LLA_F32, rho=rho, stats=stats,
                     kv_heads=Hkv, stream=stream_ptr())
    gq = torch.full((B, H, n, d), float("nan"), dtype=torch.float32, device="cuda")
    gk = torch.full((B, Hkv, n, d), float("nan"), dtype=torch.float32, device="cuda")
    gv = torch.full((B, Hkv, n, d), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = L.lla_backward_workspace_bytes(B, H, n, d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    L.lla_backward_ex(dq_, dk_, dv_, out, dg, rho, stats, gq, gk, gv, B, H, n, d, w.scale, w.lam, workspace=ws,
                      workspace_bytes=nbytes, impl=impl, kv_heads=Hkv, stream=stream_ptr())
    torch.cuda.synchronize()
    for name, a, r in (("dq", gq, rq), ("dk", gk, rk), ("dv", gv, rv)):
        err = grad_err(a.cpu().numpy().astype(np.float64), r)
        assert err.max() <= TOL, (name, float(err.max()))


@pytest.mark.parametrize("d,n,window", [(64, 700, 200), (64, 520, 96), (128, 600, 256)])
def test_backward_sliding_window(backward_oracle, d, n, window):
    # the gradient of the forward with a causal sliding window (the variant the paper's discussion suggests): the
    # query tiles start at the block of their first visible key, the key tiles stop at their last viewer
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=n, d=d, dv=d, seed=290 + d)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    ref = backward_oracle.backward(q, k, v, g, w.scale, w.lam, window=window)
    got = run_backward(w, q, k, v, g, window=window)
    for name, a, b in zip(("dq", "dk", "dv"), got, ref):
        assert np.isfinite(a).all(), name
        err = grad_err(a, b)
        assert err.max() <= TOL, (name, float(err.max()), int(err.argmax()))
    full = backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    assert grad_err(got[1], full[1]).max() > 10 * TOL        # (the window matters at these sizes)


@pytest.mark.parametrize("cfg", [3, 4])
def test_backward_full_size_sampled(backward_oracle, cfg):
    # the n = 4096 and n = 16384 workloads at full size, in the launch configuration bench.py times.  The oracle
    # cannot form whole gradients there; it checks what it can compute row by row -- dq on sampled rows, and dk, dv of
    # the last keys (which only the last rows see) -- and two identities hold at any size: sum_j dV_j = sum_i g_i
    # (the coefficients of a row sum to one) and <dV, V> = <g, o> (the output is linear in the values).
    w = inputs.CONFIGS[cfg]
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    dq_, dk_, dv_, dg = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16"), dev(g, "f32")
    shape = (w.B, w.H, w.n, w.d)
    out, rho = (torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(2))
    stats = torch.empty((w.B, w.H, w.n, 3), dtype=torch.float32, device="cuda")
    fws = torch.empty(max(L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.d), 256), dtype=torch.uint8, device="cuda")
    L.lla_forward_ex(dq_, dk_, dv_, out, w.B, w.H, w.n, w.d, w.d, w.scale, w.lam, out_dtype=L.LLA_F32, rho=rho, stats=stats,
                     workspace=fws, workspace_bytes=fws.numel(), stream=stream_ptr())
    grads = [torch.full(shape, float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    nbytes = L.lla_backward_workspace_bytes(w.B, w.H, w.n, w.d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    L.lla_backward_ex(dq_, dk_, dv_, out, dg, rho, stats, *grads, w.B, w.H, w.n, w.d, w.scale, w.lam, device_status=status,
                      workspace=ws, workspace_bytes=nbytes, stream=stream_ptr())
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert st[L.STATUS_BAD_PIVOT] == 0 and st[L.STATUS_TIMEOUT] == 0 and st[L.STATUS_ROWS_AT_CAP] == 0
    gq, gk, gv = (t.cpu().numpy().astype(np.float64) for t in grads)
    o = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(gq).all() and np.isfinite(gk).all() and np.isfinite(gv).all()
    # identities, per head
    sum_dv, sum_g = gv.sum(axis=2), g.astype(np.float64).sum(axis=2)
    assert np.abs(sum_dv - sum_g).max() <= 1e-3 * np.abs(g).sum(axis=2).max()
    lhs = (gv * v.astype(np.float64)).sum(axis=(2, 3))
    rhs = (g.astype(np.float64) * o).sum(axis=(2, 3))
    scale_ = np.sqrt((g.astype(np.float64) ** 2).sum(axis=(2, 3)) * (o ** 2).sum(axis=(2, 3)))
    assert np.abs(lhs - rhs).max() <= 1e-3 * scale_.max()
    # sampled rows and the last keys of two heads
    rng = np.random.default_rng(300 + cfg)
    m = 6
    for b, h in ((0, 0), (w.B - 1, w.H - 1)):
        first = w.d + w.d // 2 - 1
        rows = np.concatenate([[first, first + 1, 2 * w.d, 4 * w.d + 3], rng.integers(first, w.n - m, size=6),
                               np.arange(w.n - m, w.n)])
        rq, rk, rv = backward_oracle.backward_rows(q[b, h], k[b, h], v[b, h], g[b, h], w.scale, w.lam, rows)
        med = np.median(np.linalg.norm(gq[b, h], axis=1))
        err = np.linalg.norm(gq[b, h][rows] - rq, axis=1) / np.maximum(np.linalg.norm(rq, axis=1), 0.1 * med)
        assert err.max() <= TOL, ("dq", b, h, float(err.max()), int(rows[err.argmax()]))
        # only the last m rows see the last m keys: drop the other sampled rows' shares by recomputing with those rows alone
        _, tk, tv = backward_oracle.backward_rows(q[b, h], k[b, h], v[b, h], g[b, h], w.scale, w.lam, np.arange(w.n - m, w.n))
        for name, got, ref in (("dk", gk[b, h], tk), ("dv", gv[b, h], tv)):
            medk = np.median(np.linalg.norm(got, axis=1))
            e = np.linalg.norm(got[w.n - m:] - ref[w.n - m:], axis=1) / np.maximum(np.linalg.norm(ref[w.n - m:], axis=1), 0.1 * medk)
            assert e.max() <= TOL, (name, b, h, float(e.max()))


@pytest.mark.parametrize("d,n,per_head", [(64, 700, True), (64, 1024, False), (128, 600, True)])
def test_backward_block_sparse(backward_oracle, d, n, per_head):
    # the gradient of the block-sparse forward: a random mask over [query tiles of 128] x [key blocks of 64] (about
    # 40 % kept), the blocks of the first head_rows keys and each tile's diagonal blocks attended whatever it says.
    # The oracle gets the resulting row-by-key visibility.
    B, H = 1, 2
    w = inputs.CONFIGS[2].shrink(B=B, H=H, n=n, d=d, dv=d, seed=310 + d)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    tiles, blocks = (n + 127) // 128, (n + 63) // 64
    rng = np.random.default_rng(17)
    units = B * H if per_head else 1
    mask = (rng.random((units, tiles, blocks)) < 0.4).astype(np.uint8)
    head_rows = d + d // 2
    visible = np.zeros((B * H, n, n), dtype=bool)
    for u in range(B * H):
        for t in range(tiles):
            for c in range(blocks):
                if mask[u if per_head else 0, t, c] or c * 64 < head_rows or c * 64 + 63 >= t * 128:
                    visible[u, t * 128:(t + 1) * 128, c * 64:(c + 1) * 64] = True
    ref = backward_oracle.backward(q, k, v, g, w.scale, w.lam, visible=visible)
    got = run_backward(w, q, k, v, g, block_mask=torch.from_numpy(mask).cuda(),
                       block_mask_stride=tiles * blocks if per_head else 0)
    for name, a, b in zip(("dq", "dk", "dv"), got, ref):
        assert np.isfinite(a).all(), name
        err = grad_err(a, b)
        assert err.max() <= TOL, (name, float(err.max()), int(err.argmax()))
    dense = backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    assert grad_err(got[1], dense[1]).max() > 10 * TOL        # (the mask matters)


@pytest.mark.parametrize("d,n,nq,window,Hkv", [(64, 700, 300, 0, 0), (64, 300, 260, 0, 0), (128, 640, 200, 0, 0),
                                                (64, 900, 500, 256, 2)])
def test_backward_chunk_of_queries(backward_oracle, d, n, nq, window, Hkv):
    # the gradient of a forward that had only the queries of the last nq positions (q_rows): dq has nq rows, dk and dv
    # all n.  Cases: the chunk starts beyond the directly-solved positions; it starts among them (some of its rows
    # are solved directly); d = 128; with a sliding window and grouped key/value heads on top.
    B, H = 1, 2
    w = inputs.CONFIGS[2].shrink(B=B, H=H, n=n, d=d, dv=d, seed=320 + d + nq)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    off = n - nq
    qc, gc = q[:, :, off:], g[:, :, off:]
    if Hkv:
        grp = H // Hkv
        k, v = k[:, :Hkv], v[:, :Hkv]
        rq, rk, rv = backward_oracle.backward(qc, np.repeat(k, grp, axis=1), np.repeat(v, grp, axis=1), gc, w.scale, w.lam,
                                              window=window)
        rk = rk.reshape(B, Hkv, grp, n, d).sum(axis=2)
        rv = rv.reshape(B, Hkv, grp, n, d).sum(axis=2)
    else:
        rq, rk, rv = backward_oracle.backward(qc, k, v, gc, w.scale, w.lam, window=window)
    dq_, dk_, dv_, dg = dev(qc, "bf16"), dev(k, "bf16"), dev(v, "bf16"), dev(gc, "f32")
    out = torch.empty((B, H, nq, d), dtype=torch.float32, device="cuda")
    rho = torch.empty((B, H, nq, d), dtype=torch.float32, device="cuda")
    stats = torch.empty((B, H, nq, 3), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq_, dk_, dv_, out, B, H, n, d, d, w.scale, w.lam, out_dtype=L.LLA_F32, rho=rho, stats=stats,
                     q_rows=nq, window=window, kv_heads=Hkv, stream=stream_ptr())
    gq = torch.full((B, H, nq, d), float("nan"), dtype=torch.float32, device="cuda")
    gk = torch.full(k.shape, float("nan"), dtype=torch.float32, device="cuda")
    gv = torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda")
    nbytes = L.lla_backward_workspace_bytes(B, H, n, d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
    L.lla_backward_ex(dq_, dk_, dv_, out, dg, rho, stats, gq, gk, gv, B, H, n, d, w.scale, w.lam, device_status=status,
                      workspace=ws, workspace_bytes=nbytes, q_rows=nq, window=window, kv_heads=Hkv, stream=stream_ptr())
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert st[L.STATUS_BAD_PIVOT] == 0 and st[L.STATUS_TIMEOUT] == 0
    for name, a, r in (("dq", gq, rq), ("dk", gk, rk), ("dv", gv, rv)):
        a = a.cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all(), name
        err = grad_err(a, r)
        assert err.max() <= TOL, (name, float(err.max()), int(err.argmax()))


def test_backward_bounded_waits_run_out_and_the_context_stays_usable(backward_oracle):
    # Failure detection without a fault, as in the forward: the copy-issuing warps of the solve and of the three
    # tensor-core kernels issue nothing, so every bounded wait runs out (cap 2^20 clocks) with no copy or MMA in
    # flight; the blocks release their tensor memory and leave, the status words count them, the call returns
    # normally, and the next calls on the same context are correct.
    w = inputs.CONFIGS[2].shrink(B=1, H=1, n=256, seed=330)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    ref = backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    dq_, dk_, dv_, dg = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16"), dev(g, "f32")
    shape = (1, 1, w.n, w.d)
    out, rho = (torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(2))
    stats = torch.empty((1, 1, w.n, 3), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq_, dk_, dv_, out, 1, 1, w.n, w.d, w.d, w.scale, w.lam, out_dtype=L.LLA_F32, rho=rho, stats=stats,
                     stream=stream_ptr())
    nbytes = L.lla_backward_workspace_bytes(1, 1, w.n, w.d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")

    def run(**kw):
        grads = [torch.full(shape, float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
        L.lla_backward_ex(dq_, dk_, dv_, out, dg, rho, stats, *grads, 1, 1, w.n, w.d, w.scale, w.lam, device_status=status,
                          workspace=ws, workspace_bytes=nbytes, stream=stream_ptr(), **kw)
        torch.cuda.synchronize()
        return [t.cpu().numpy().astype(np.float64) for t in grads], status.cpu().tolist()

    _, st = run(debug_wait_clocks=1 << 20, debug_flags=L.LLA_DEBUG_NO_LOADS)
    # two query tiles in each of the moments, solve and dQ kernels, two key tiles in the dK/dV kernel
    assert st[L.STATUS_TIMEOUT] == 8
    for _ in range(2):
        grads, st = run()
        assert st[L.STATUS_TIMEOUT] == 0
        for name, a, b in zip(("dq", "dk", "dv"), grads, ref):
            assert grad_err(a, b).max() <= TOL, name


def test_backward_with_preconditioned_solve(backward_oracle):
    w = inputs.CONFIGS[2].shrink(B=1, H=2, n=640, seed=295)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    ref = backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    its = [torch.full((w.B, w.H, w.n), -1, dtype=torch.int32, device="cuda") for _ in range(2)]
    plain = run_backward(w, q, k, v, g, iters=its[0])
    got = run_backward(w, q, k, v, g, iters=its[1], cg_precondition=1)
    for name, a, b in zip(("dq", "dk", "dv"), got, ref):
        assert grad_err(a, b).max() <= TOL, name
    a, b = (t.cpu().numpy().ravel() for t in its)
    assert b[b >= 0].mean() < 0.75 * a[a >= 0].mean()        # fewer iterations of the extra solve


def test_backward_dq_is_bit_identical_between_runs():
    # dq comes from plain stores of the query tile that owns the rows (and of one block per directly-solved row), so
    # two runs give the same bits; dk and dv are summed atomically and only agree to rounding
    w = inputs.CONFIGS[2].shrink(B=2, H=4, seed=280)
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    a = run_backward(w, q, k, v, g)
    b = run_backward(w, q, k, v, g)
    assert np.array_equal(a[0], b[0])
    for x, y in zip(a[1:], b[1:]):
        assert np.abs(x - y).max() <= 1e-5 * np.abs(x).max()


def test_backward_window_argument_checks():
    ok = 0x1000
    ws = torch.empty(L.lla_backward_workspace_bytes(1, 1, 256, 64), dtype=torch.uint8, device="cuda")
    for kw in (dict(window=50), dict(window=128, impl=L.LLA_IMPL_SIMT)):      # below head_rows; CUDA-core kernels
        with pytest.raises(L.LlaError) as e:
            L.lla_backward_ex(ok, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1, 1, 256, 64, 0.125, 1e-3, workspace=ws,
                              workspace_bytes=ws.numel(), **kw)
        assert e.value.status == 2


def test_backward_argument_checks():
    ok = 0x1000
    with pytest.raises(L.LlaError) as e:
        L.lla_backward_ex(ok, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1, 1, 64, 64, 0.125, 1e-3)
    assert e.value.status == 3                       # no workspace
    with pytest.raises(L.LlaError) as e:
        L.lla_backward_ex(ok, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1, 1, 64, 16, 0.25, 1e-3)
    assert e.value.status == 2                       # head size
    with pytest.raises(L.LlaError) as e:
        L.lla_backward_ex(None, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1, 1, 64, 64, 0.125, 1e-3)
    assert e.value.status == 1
