"""Pins for the gradient oracle (oracle/lla_backward_oracle.py): everything here is fixed by the paper or
by mathematics, none of it by the CUDA path.

  (a) central finite differences of the separate C forward oracle (different code, different solver)
  (b) the forward the gradient differentiates equals the C oracle's forward
  (c) sum_j s_ij = 1  =>  sum_j dV_j = sum_i g_i;   v -> v + c leaves dQ, dK unchanged
  (d) lambda -> infinity: the gradient tends to the textbook softmax-attention gradient, error ~ 1/lambda
  (e) a single token: o_0 = v_0 for every lambda > 0, so dQ = dK = 0 and dV = g
  (f) the hand-derived formulas of the paper's backward appendix, evaluated literally in numpy
  (g) sliding window: the windowed forward is the C oracle's forward of each row's own key range, and the windowed
      gradient is the finite difference of that
  (h) sparse visibility: the same with an arbitrary set of visible keys per row (the C oracle's decode entry point
      on exactly those keys)
"""
import numpy as np
import pytest

from oracle import lla_backward_oracle as bwd
from oracle import lla_oracle as fwd_c


def _inputs(seed, n, d, dv, B=1, H=1):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, H, n, d)) / np.sqrt(d)
    k = rng.standard_normal((B, H, n, d)) / np.sqrt(d)
    v = rng.standard_normal((B, H, n, dv))
    g = rng.standard_normal((B, H, n, dv))
    return q, k, v, g


def test_forward_of_gradient_oracle_equals_c_oracle():
    q, k, v, _ = _inputs(1, 40, 8, 5)
    a = bwd.forward(q, k, v, 0.35, 1e-2)
    b = fwd_c.forward(q, k, v, 0.35, 1e-2)
    assert np.abs(a - b).max() <= 1e-9 * np.abs(b).max()


@pytest.mark.parametrize("causal", [True, False])
def test_finite_differences_of_c_forward_oracle(causal):
    n, d, dv, scale, lam = 7, 3, 2, 0.6, 5e-2
    q, k, v, g = _inputs(2, n, d, dv)
    dq, dk, dv_ = bwd.backward(q, k, v, g, scale, lam, causal=causal)

    def loss(q_, k_, v_):
        return float((fwd_c.forward(q_, k_, v_, scale, lam, causal=causal) * g).sum())

    eps = 1e-5
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv_)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            args_p = {"q": q, "k": k, "v": v, name: xp}
            args_m = {"q": q, "k": k, "v": v, name: xm}
            num[idx] = (loss(args_p["q"], args_p["k"], args_p["v"]) - loss(args_m["q"], args_m["k"], args_m["v"])) / (2 * eps)
        assert np.abs(num - grad).max() <= 2e-7 * max(1.0, np.abs(grad).max()), name


def test_value_gradient_sums_and_shift_invariance():
    q, k, v, g = _inputs(3, 48, 6, 4, B=1, H=2)
    dq, dk, dv = bwd.backward(q, k, v, g, 0.4, 1e-2)
    assert np.abs(dv.sum(axis=2) - g.sum(axis=2)).max() <= 1e-9
    dq2, dk2, _ = bwd.backward(q, k, v + 3.0, g, 0.4, 1e-2)
    assert np.abs(dq2 - dq).max() <= 1e-8 * np.abs(dq).max()
    assert np.abs(dk2 - dk).max() <= 1e-8 * np.abs(dk).max()


def _softmax_attention_grad(q, k, v, g, scale):
    n = q.shape[0]
    s = scale * q @ k.T
    s = np.where(np.tril(np.ones((n, n), bool)), s, -np.inf)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    o = p @ v
    ds = p * (g @ v.T - (g * o).sum(axis=1, keepdims=True))
    return scale * ds @ k, scale * ds.T @ q, p.T @ g


def test_large_ridge_limit_is_softmax_attention_gradient():
    q, k, v, g = _inputs(4, 24, 4, 3)
    ref = _softmax_attention_grad(q[0, 0], k[0, 0], v[0, 0], g[0, 0], 0.5)
    errs = []
    for lam in (1e4, 1e6):
        got = bwd.backward(q, k, v, g, 0.5, lam)
        errs.append(max(np.abs(a[0, 0] - b).max() for a, b in zip(got, ref)))
    assert errs[0] < 1e-2 and errs[1] < 1e-4 and errs[1] < 0.02 * errs[0]


def test_single_token():
    q, k, v, g = _inputs(5, 1, 4, 3)
    dq, dk, dv = bwd.backward(q, k, v, g, 0.5, 1e-3)
    assert np.abs(dq).max() <= 1e-12 and np.abs(dk).max() <= 1e-12
    assert np.abs(dv - g).max() <= 1e-12


def _appendix_formulas(q, k, v, g, scale, lam):
    """Backward appendix, literally: gamma, beta, c, u, Delta_mu, dL/dSigma, dL/dw, dL/dz, then the
    chain rule to k_j and q_i.  Raw weights exp(scale q.k), ridge lam (no max shift)."""
    n, d = q.shape
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for i in range(n):
        K, V = k[: i + 1], v[: i + 1]
        Z = K - q[i]
        w = np.exp(scale * K @ q[i])
        omega, mu = w.sum(), w @ Z
        Sigma = (Z * w[:, None]).T @ Z + lam * np.eye(d)
        rho = np.linalg.solve(Sigma, mu)
        delta = omega - mu @ rho
        nij = 1.0 - Z @ rho
        s = w * nij / delta
        gamma = V @ g[i]
        beta = (gamma * s).sum() / delta
        c = gamma * w / delta
        u = np.linalg.solve(Sigma, c @ Z)
        dmu = -u + 2.0 * beta * rho
        dSigma = -0.5 * np.outer(rho, dmu) + 0.5 * np.outer(u, rho)
        dw = gamma * nij / delta - beta + Z @ dmu + np.einsum("jc,ce,je->j", Z, dSigma, Z)
        dz = -np.outer(c, rho) + np.outer(w, dmu) + 2.0 * w[:, None] * (Z @ dSigma.T)
        dv[: i + 1] += np.outer(s, g[i])
        dk[: i + 1] += (dw * w * scale)[:, None] * q[i] + dz
        dq[i] += (dw * w * scale) @ K - dz.sum(axis=0)
    return dq, dk, dv


def test_backward_appendix_formulas():
    q, k, v, g = _inputs(6, 20, 5, 4)
    got = bwd.backward(q, k, v, g, 0.45, 2e-2)
    ref = _appendix_formulas(q[0, 0], k[0, 0], v[0, 0], g[0, 0], 0.45, 2e-2)
    for a, b in zip(got, ref):
        assert np.abs(a[0, 0] - b).max() <= 1e-9 * max(1.0, np.abs(b).max())


def test_ridge_gradient_by_finite_differences_of_c_oracle():
    # d loss / d lambda_i for a ridge of its own per query row: the C forward oracle takes per-row ridges
    n, d, dv, scale, lam = 9, 3, 2, 0.6, 5e-2
    q, k, v, g = _inputs(7, n, d, dv)
    *_, dlam = bwd.backward(q, k, v, g, scale, lam, want_dlambda=True)
    eps = 1e-6
    for i in range(n):
        lp = np.full((1, 1, n), lam)
        lm = lp.copy()
        lp[0, 0, i] += eps
        lm[0, 0, i] -= eps
        num = float(((fwd_c.forward(q, k, v, scale, lp) - fwd_c.forward(q, k, v, scale, lm)) * g).sum()) / (2 * eps)
        assert abs(num - dlam[0, 0, i]) <= 1e-6 * max(1.0, abs(num)), i
    # the first row's output is v_0 for every positive ridge: no dependence on lambda
    assert abs(dlam[0, 0, 0]) <= 1e-12


def _windowed_forward_by_c_oracle(q, k, v, scale, lam, window):
    """Row i of a sliding-window forward is the last row of a plain causal forward over keys i - window + 1 .. i
    alone (the C oracle knows no window): the definition of the window, evaluated row by row."""
    B, H, n, _ = q.shape
    out = np.zeros(v.shape)
    for i in range(n):
        lo = max(0, i - window + 1)
        sl = slice(lo, i + 1)
        qq = np.repeat(q[:, :, i:i + 1], i + 1 - lo, axis=2)          # only the last row's query matters
        out[:, :, i] = fwd_c.forward(qq, k[:, :, sl], v[:, :, sl], scale, lam)[:, :, -1]
    return out


def test_sliding_window_forward_and_finite_differences():
    n, d, dv, scale, lam, window = 9, 3, 2, 0.6, 5e-2, 4
    q, k, v, g = _inputs(8, n, d, dv)
    ref = _windowed_forward_by_c_oracle(q, k, v, scale, lam, window)
    assert np.abs(bwd.forward(q, k, v, scale, lam, window=window) - ref).max() <= 1e-9 * np.abs(ref).max()
    assert np.abs(bwd.forward(q, k, v, scale, lam, window=n) - bwd.forward(q, k, v, scale, lam)).max() == 0.0
    dq, dk, dv_ = bwd.backward(q, k, v, g, scale, lam, window=window)
    full = bwd.backward(q, k, v, g, scale, lam)
    assert np.abs(dk - full[1]).max() > 1e-3          # the window changes the gradient (the pin below is not vacuous)

    def loss(q_, k_, v_):
        return float((_windowed_forward_by_c_oracle(q_, k_, v_, scale, lam, window) * g).sum())

    eps = 1e-5
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv_)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            ap = {"q": q, "k": k, "v": v, name: xp}
            am = {"q": q, "k": k, "v": v, name: xm}
            num[idx] = (loss(ap["q"], ap["k"], ap["v"]) - loss(am["q"], am["k"], am["v"])) / (2 * eps)
        assert np.abs(num - grad).max() <= 2e-7 * max(1.0, np.abs(grad).max()), name


def test_row_shares_add_up_to_the_gradient():
    # backward_rows (one row at a time, for the full-size tests) against backward on a small case: all rows' shares
    # sum to the gradient, and the last m rows alone give the complete dk, dv of the last m keys
    n, d, dv, scale, lam = 24, 5, 3, 0.5, 2e-2
    q, k, v, g = _inputs(9, n, d, dv)
    dq, dk, dv_ = (x[0, 0] for x in bwd.backward(q, k, v, g, scale, lam))
    rq, rk, rv = bwd.backward_rows(q[0, 0], k[0, 0], v[0, 0], g[0, 0], scale, lam, range(n))
    for a, b in ((rq, dq), (rk, dk), (rv, dv_)):
        assert np.abs(a - b).max() <= 1e-12 * max(1.0, np.abs(b).max())
    m = 5
    rq, rk, rv = bwd.backward_rows(q[0, 0], k[0, 0], v[0, 0], g[0, 0], scale, lam, range(n - m, n))
    assert np.abs(rq - dq[n - m:]).max() <= 1e-12 * np.abs(dq).max()
    assert np.abs(rk[n - m:] - dk[n - m:]).max() <= 1e-12 * np.abs(dk).max()
    assert np.abs(rv[n - m:] - dv_[n - m:]).max() <= 1e-12 * np.abs(dv_).max()
    assert np.abs(rk[:n - m] - dk[:n - m]).max() > 1e-3      # (the earlier keys also hear from the other rows)


def _sparse_forward_by_c_oracle(q, k, v, scale, lam, visible):
    """Row i of a forward with a visibility matrix is a single query over exactly its visible keys: the C oracle's
    decode entry point, which knows no mask, on those keys."""
    B, H, n, d = q.shape
    out = np.zeros(v.shape)
    for i in range(n):
        idx = np.nonzero(visible[i, :i + 1])[0]
        kc = np.zeros((B, H, n, d))
        vc = np.zeros((B, H, n, v.shape[3]))
        kc[:, :, :len(idx)] = k[:, :, idx]
        vc[:, :, :len(idx)] = v[:, :, idx]
        out[:, :, i] = fwd_c.decode(q[:, :, i], kc, vc, np.full(B, len(idx), dtype=np.int32), scale, lam)
    return out


def test_sparse_visibility_forward_and_finite_differences():
    n, d, dv, scale, lam = 9, 3, 2, 0.6, 5e-2
    q, k, v, g = _inputs(10, n, d, dv)
    rng = np.random.default_rng(11)
    visible = rng.random((n, n)) < 0.6
    visible[np.arange(n), np.arange(n)] = True           # every row keeps its own key
    ref = _sparse_forward_by_c_oracle(q, k, v, scale, lam, visible)
    assert np.abs(bwd.forward(q, k, v, scale, lam, visible=visible) - ref).max() <= 1e-9 * np.abs(ref).max()
    dq, dk, dv_ = bwd.backward(q, k, v, g, scale, lam, visible=visible)

    def loss(q_, k_, v_):
        return float((_sparse_forward_by_c_oracle(q_, k_, v_, scale, lam, visible) * g).sum())

    eps = 1e-5
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv_)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            ap = {"q": q, "k": k, "v": v, name: xp}
            am = {"q": q, "k": k, "v": v, name: xm}
            num[idx] = (loss(ap["q"], ap["k"], ap["v"]) - loss(am["q"], am["k"], am["v"])) / (2 * eps)
        assert np.abs(num - grad).max() <= 2e-7 * max(1.0, np.abs(grad).max()), name


def test_chunk_of_queries_is_the_full_gradient_with_zero_upstream_elsewhere():
    # the last nq queries against all n keys: the loss of the whole sequence with g = 0 on the earlier rows
    n, nq, d, dv, scale, lam = 20, 7, 4, 3, 0.5, 3e-2
    q, k, v, g = _inputs(12, n, d, dv)
    g0 = g.copy()
    g0[:, :, :n - nq] = 0.0
    fq, fk, fv = bwd.backward(q, k, v, g0, scale, lam)
    cq, ck, cv = bwd.backward(q[:, :, n - nq:], k, v, g[:, :, n - nq:], scale, lam)
    assert cq.shape == (1, 1, nq, d)
    assert np.abs(cq - fq[:, :, n - nq:]).max() <= 1e-12 * np.abs(fq).max()
    assert np.abs(ck - fk).max() <= 1e-12 * np.abs(fk).max()
    assert np.abs(cv - fv).max() <= 1e-12 * np.abs(fv).max()
    assert np.abs(fq[:, :, :n - nq]).max() == 0.0
