"""Pins for the float64 CPU oracle: every check here is something the paper's definition or the
mathematics fixes, computed by a route other than the oracle's own code.

The paper prints no numeric example of an LLA output, so the pins are: brute-force weighted
least squares of the local-linear objective (Section 2.3, Eq. "lla_obj"), a library ridge
regression with sample weights, closed forms (first row, hand-worked d=1 case), the softmax /
Nadaraya-Watson limit (Eq. "local_constant"), affine reproduction, shift equivariance,
permutation invariance, the dual (Gram) form and the decomposition of Eq. "lla_decomp".
"""
import json
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(seed, B, H, n, d, dv, kscale=None):
    rng = np.random.default_rng(seed)
    s = 1.0 / np.sqrt(d) if kscale is None else kscale
    q = rng.standard_normal((B, H, n, d)) * s
    k = rng.standard_normal((B, H, n, d)) * s
    v = rng.standard_normal((B, H, n, dv))
    return q, k, v


def _wls_intercept(qi, K, V, scale, lam):
    """Brute force: minimise 1/2 sum_j w_j |v_j - b - W z_j|^2 + lam/2 |W|_F^2 over (b, W) by
    stacking sqrt-weighted data rows and sqrt(lam) ridge rows into one dense least-squares
    problem; raw weights exp(scale q.k), no max subtraction."""
    L, d = K.shape
    w = np.exp(scale * (K @ qi))
    Z = K - qi
    A = np.zeros((L + d, 1 + d))
    Y = np.zeros((L + d, V.shape[1]))
    A[:L, 0] = np.sqrt(w)
    A[:L, 1:] = np.sqrt(w)[:, None] * Z
    Y[:L] = np.sqrt(w)[:, None] * V
    A[L:, 1:] = np.sqrt(lam) * np.eye(d)
    sol, *_ = np.linalg.lstsq(A, Y, rcond=None)
    return sol[0]


def _softmax_rows(q, k, v, scale):
    B, H, n, _ = q.shape
    out = np.zeros(v.shape)
    for b in range(B):
        for h in range(H):
            s = scale * q[b, h] @ k[b, h].T
            s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[b, h] = p @ v[b, h]
    return out


def test_brute_force_wls_tiny(oracle):
    # brute force on tiny inputs: n <= 8, every causal row equals the intercept of a dense WLS fit.
    for seed, (n, d, dv, scale, lam) in enumerate([(8, 3, 2, 0.7, 0.05), (6, 2, 4, 3.0, 1e-3),
                                                   (8, 4, 3, 1.5, 0.3), (5, 1, 1, 2.0, 0.01)]):
        q, k, v = _rand(seed, 2, 2, n, d, dv, kscale=1.0)
        out = oracle.forward(q, k, v, scale, lam, causal=True)
        for b in range(2):
            for h in range(2):
                for i in range(n):
                    ref = _wls_intercept(q[b, h, i], k[b, h, :i + 1], v[b, h, :i + 1], scale, lam)
                    np.testing.assert_allclose(out[b, h, i], ref, rtol=1e-8, atol=1e-10)


def test_wls_with_large_scores_checks_ridge_rescaling(oracle):
    # Scores up to ~+-25: the oracle evaluates exp(s - m) and must rescale the ridge by exp(-m).
    # The brute force uses raw weights, so a missing or wrong rescale shows up here.
    q, k, v = _rand(11, 1, 1, 8, 3, 2, kscale=1.0)
    scale, lam = 6.0, 0.5
    out = oracle.forward(q, k, v, scale, lam)
    smax = np.abs(scale * q[0, 0] @ k[0, 0].T).max()
    assert smax > 8.0
    for i in range(8):
        ref = _wls_intercept(q[0, 0, i], k[0, 0, :i + 1], v[0, 0, :i + 1], scale, lam)
        np.testing.assert_allclose(out[0, 0, i], ref, rtol=1e-8, atol=1e-10)


def test_library_weighted_ridge(oracle):
    # LLA at q is the intercept of ridge regression on features k_j - q with sample weights w_j
    # and an unpenalised intercept; scikit-learn's Ridge minimises sum w|y - Xb - c|^2 + alpha|b|^2.
    from sklearn.linear_model import Ridge
    n, d, dv, scale, lam = 40, 6, 3, 1.3, 0.02
    q, k, v = _rand(5, 1, 2, n, d, dv, kscale=0.8)
    out = oracle.forward(q, k, v, scale, lam)
    for h in range(2):
        for i in (0, 1, 5, 17, 39):
            K, V, qi = k[0, h, :i + 1], v[0, h, :i + 1], q[0, h, i]
            w = np.exp(scale * K @ qi)
            model = Ridge(alpha=lam, fit_intercept=True, solver="cholesky").fit(K - qi, V, sample_weight=w)
            np.testing.assert_allclose(out[0, h, i], model.intercept_, rtol=1e-8, atol=1e-10)


def test_uniform_weights_reduce_to_plain_ridge(oracle):
    # scale = 0 -> every weight is 1: ordinary ridge regression on the prefix, predicted at q.
    from sklearn.linear_model import Ridge
    n, d, dv, lam = 30, 5, 2, 0.1
    q, k, v = _rand(6, 1, 1, n, d, dv, kscale=1.0)
    out = oracle.forward(q, k, v, 0.0, lam)
    for i in (3, 10, 29):
        model = Ridge(alpha=lam, fit_intercept=True, solver="cholesky").fit(k[0, 0, :i + 1], v[0, 0, :i + 1])
        pred = model.predict(q[0, 0, i][None])[0]
        np.testing.assert_allclose(out[0, 0, i], pred, rtol=1e-9, atol=1e-11)


def test_softmax_limit(oracle):
    # (a): lambda -> infinity kills the slope, leaving the Nadaraya-Watson / softmax average;
    # the gap decays like 1/lambda.
    q, k, v = _rand(1, 1, 2, 48, 8, 8)
    scale = 1.0 / np.sqrt(8)
    ref = _softmax_rows(q, k, v, scale)
    errs = []
    for lam in (1e2, 1e4, 1e6, 1e8):
        out = oracle.forward(q, k, v, scale, lam)
        errs.append(np.abs(out - ref).max())
    assert errs[0] < 0.2 and errs[-1] < 1e-6
    for a, b in zip(errs, errs[1:]):
        assert b < a * 0.02           # ~100x per step of 100x in lambda


def test_affine_reproduction_at_zero_ridge(oracle):
    # (b): v_j = A k_j + c exactly, lambda = 0, at least d+2 visible keys -> output A q_i + c.
    rng = np.random.default_rng(2)
    n, d, dv = 24, 4, 3
    q, k, _ = _rand(2, 1, 1, n, d, dv, kscale=1.0)
    A = rng.standard_normal((dv, d))
    c = rng.standard_normal(dv)
    v = k @ A.T + c
    out = oracle.forward(q, k, v, 0.9, 0.0)
    want = q @ A.T + c
    np.testing.assert_allclose(out[0, 0, d + 1:], want[0, 0, d + 1:], rtol=1e-8, atol=1e-9)
    # with a ridge the slope is shrunk, so the reproduction must NOT be exact
    out_r = oracle.forward(q, k, v, 0.9, 1.0)
    assert np.abs(out_r[0, 0, d + 1:] - want[0, 0, d + 1:]).max() > 1e-3


def test_shift_equivariance_and_linearity_in_v(oracle):
    # (c): adding a constant vector to every value shifts every output by it; outputs are linear in V.
    q, k, v = _rand(3, 2, 2, 20, 5, 4)
    rng = np.random.default_rng(33)
    c = rng.standard_normal(4)
    v2 = rng.standard_normal(v.shape)
    scale, lam = 0.6, 0.03
    o1 = oracle.forward(q, k, v, scale, lam)
    np.testing.assert_allclose(oracle.forward(q, k, v + c, scale, lam), o1 + c, rtol=0, atol=1e-11)
    o2 = oracle.forward(q, k, v2, scale, lam)
    np.testing.assert_allclose(oracle.forward(q, k, 2.0 * v - 3.0 * v2, scale, lam),
                               2.0 * o1 - 3.0 * o2, rtol=0, atol=1e-10)


def test_first_row_is_its_own_value(oracle):
    # One visible pair: rho = w z/(lam + w|z|^2), the single coefficient cancels -> o_0 = v_0.
    q, k, v = _rand(4, 2, 3, 5, 6, 7)
    for lam in (1e-3, 1.0, 50.0):
        out = oracle.forward(q, k, v, 0.4, lam)
        np.testing.assert_allclose(out[:, :, 0], v[:, :, 0], rtol=1e-12, atol=1e-13)


def test_hand_worked_cases(oracle):
    # Closed forms derived by hand from Eq. "lla" for d = 1 (see the fixture's "derivation").
    with open(os.path.join(GOLDEN, "hand_worked_d1.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        q = np.array(c["q"], dtype=np.float64).reshape(1, 1, -1, 1)
        k = np.array(c["k"], dtype=np.float64).reshape(1, 1, -1, 1)
        v = np.array(c["v"], dtype=np.float64).reshape(1, 1, -1, 1)
        out = oracle.forward(q, k, v, c["scale"], c["lambda"], causal=True)
        np.testing.assert_allclose(out[0, 0, :, 0], np.array(c["out"], dtype=np.float64),
                                   rtol=1e-13, atol=1e-14)


def test_dual_gram_form(oracle):
    # Independent algebra: with Z the centred keys, alpha = (Z Z^T + lam diag(1/w))^{-1} 1 gives
    # w_j (1 - z_j^T rho) = lam alpha_j, hence o = sum alpha_j v_j / sum alpha_j.
    q, k, v = _rand(7, 1, 1, 12, 5, 3, kscale=1.0)
    scale, lam = 0.8, 0.07
    out = oracle.forward(q, k, v, scale, lam)
    for i in range(12):
        K, V, qi = k[0, 0, :i + 1], v[0, 0, :i + 1], q[0, 0, i]
        w = np.exp(scale * K @ qi)
        Z = K - qi
        alpha = np.linalg.solve(Z @ Z.T + lam * np.diag(1.0 / w), np.ones(i + 1))
        np.testing.assert_allclose(out[0, 0, i], alpha @ V / alpha.sum(), rtol=1e-9, atol=1e-11)


def test_decomposition_with_optimal_slope(oracle):
    # Eq. "lla_decomp": b = sum_j s_j (v_j - W k_j) + W q with softmax weights s and the optimal
    # slope W = S_vk C^{-1} of the weighted, centred ridge problem.
    q, k, v = _rand(8, 1, 1, 30, 4, 3, kscale=1.0)
    scale, lam = 0.5, 0.2
    out, rho, aux, status = oracle.forward_rows(q, k, v, scale, lam, want_aux=True)
    assert (status == 0).all()
    for i in (2, 9, 29):
        K, V, qi = k[0, 0, :i + 1], v[0, 0, :i + 1], q[0, 0, i]
        w = np.exp(scale * K @ qi)
        s = w / w.sum()
        kbar, vbar = s @ K, s @ V
        C = (w[:, None] * (K - kbar)).T @ (K - kbar) + lam * np.eye(4)
        Svk = (w[:, None] * (V - vbar)).T @ (K - kbar)
        W = Svk @ np.linalg.inv(C)
        b = s @ (V - K @ W.T) + W @ qi
        np.testing.assert_allclose(out[i], b, rtol=1e-9, atol=1e-11)
        # auxiliary outputs: rho solves Sigma rho = mu, delta = omega - mu.rho (max-subtracted frame)
        m = (scale * K @ qi).max()
        wm = np.exp(scale * K @ qi - m)
        Z = K - qi
        Sigma = (wm[:, None] * Z).T @ Z + lam * np.exp(-m) * np.eye(4)
        mu = wm @ Z
        np.testing.assert_allclose(rho[i], np.linalg.solve(Sigma, mu), rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(aux[i], [m, wm.sum(), wm.sum() - mu @ rho[i]], rtol=1e-10)


def test_noncausal_permutation_invariance_and_causal_prefix(oracle):
    q, k, v = _rand(9, 1, 2, 16, 4, 4)
    scale, lam = 0.5, 0.01
    full = oracle.forward(q, k, v, scale, lam, causal=False)
    perm = np.random.default_rng(0).permutation(16)
    np.testing.assert_allclose(oracle.forward(q, k[:, :, perm], v[:, :, perm], scale, lam, causal=False),
                               full, rtol=1e-10, atol=1e-12)
    # the last causal row sees every key, so it equals the non-causal row; earlier rows do not
    causal = oracle.forward(q, k, v, scale, lam, causal=True)
    np.testing.assert_allclose(causal[:, :, -1], full[:, :, -1], rtol=1e-12, atol=1e-14)
    assert np.abs(causal[:, :, 3] - full[:, :, 3]).max() > 1e-3
    # and causal row i must not depend on later keys/values
    k2, v2 = k.copy(), v.copy()
    k2[:, :, 9:] += 1.0
    v2[:, :, 9:] -= 2.0
    np.testing.assert_array_equal(oracle.forward(q, k2, v2, scale, lam)[:, :, :9], causal[:, :, :9])


def test_decode_equals_last_prefill_row(oracle):
    rng = np.random.default_rng(10)
    B, H, Lmax, d, dv = 3, 2, 20, 4, 5
    kc = rng.standard_normal((B, H, Lmax, d))
    vc = rng.standard_normal((B, H, Lmax, dv))
    qd = rng.standard_normal((B, H, d))
    lens = np.array([20, 1, 7], dtype=np.int32)
    out = oracle.decode(qd, kc, vc, lens, 0.5, 0.02)
    for b in range(B):
        L = int(lens[b])
        qfull = np.zeros((1, H, L, d))
        qfull[0, :, L - 1] = qd[b]
        ref = oracle.forward(qfull, kc[b:b + 1, :, :L], vc[b:b + 1, :, :L], 0.5, 0.02)
        np.testing.assert_allclose(out[b], ref[0, :, L - 1], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(out[1], vc[1, :, 0], rtol=1e-12)    # one cached pair -> its value


def test_float32_inputs_match_float64_inputs(oracle):
    q, k, v = _rand(12, 1, 2, 10, 4, 4)
    q32, k32, v32 = (x.astype(np.float32) for x in (q, k, v))
    a = oracle.forward(q32, k32, v32, 0.5, 0.01)
    b = oracle.forward(q32.astype(np.float64), k32.astype(np.float64), v32.astype(np.float64), 0.5, 0.01)
    np.testing.assert_array_equal(a, b)


def test_zero_ridge_singular_row_is_flagged(oracle):
    # lambda = 0 with fewer than d+1 keys: Sigma is singular; the row must be flagged, not faked.
    q, k, v = _rand(13, 1, 1, 8, 4, 2, kscale=1.0)
    out, rho, aux, status = oracle.forward_rows(q, k, v, 0.5, 0.0, want_aux=True)
    assert status[0] == 1 and np.isnan(out[0]).all()
    assert status[7] == 0 and np.isfinite(out[7]).all()


def test_row_subset_and_threads(oracle):
    q, k, v = _rand(14, 2, 2, 12, 3, 3)
    full = oracle.forward(q, k, v, 0.5, 0.01).reshape(-1, 3)
    rows = np.array([0, 47, 13, 13, 30], dtype=np.int64)
    np.testing.assert_array_equal(oracle.forward_rows(q, k, v, 0.5, 0.01, rows=rows), full[rows])
    assert oracle.threads() >= 1


def test_per_token_ridge_matches_brute_force_row_by_row(oracle):
    # Ridge variants (the appendix on learnable, per-token regularisation): one lambda per query
    # row.  Every row must equal the dense WLS fit with that row's own ridge.
    n, d, dv, scale = 7, 3, 2, 1.2
    q, k, v = _rand(21, 2, 2, n, d, dv, kscale=1.0)
    lam = np.random.default_rng(22).uniform(1e-3, 0.5, size=(2, 2, n))
    out = oracle.forward(q, k, v, scale, lam, causal=True)
    for b in range(2):
        for h in range(2):
            for i in range(n):
                ref = _wls_intercept(q[b, h, i], k[b, h, :i + 1], v[b, h, :i + 1], scale, lam[b, h, i])
                np.testing.assert_allclose(out[b, h, i], ref, rtol=1e-8, atol=1e-10)
    # a constant array is the scalar case
    np.testing.assert_allclose(oracle.forward(q, k, v, scale, np.full((2, 2, n), 0.07)),
                               oracle.forward(q, k, v, scale, 0.07), rtol=1e-13, atol=1e-15)


def test_printed_ridge_equals_raw_frame_ridge_times_exp_max(oracle):
    # Algorithm 1/2 as printed add lambda to the moments of the max-subtracted weights exp(s - m_i).
    # Scaling all weights by c is the same problem as dividing the ridge by c, so the printed variant
    # is the definition with ridge lambda * exp(m_i): brute force with RAW weights and that ridge.
    n, d, dv, scale, lam = 8, 3, 3, 3.0, 0.02
    q, k, v = _rand(23, 1, 2, n, d, dv, kscale=1.0)
    out = oracle.forward(q, k, v, scale, lam, causal=True, ridge_mode="printed")
    plain = oracle.forward(q, k, v, scale, lam, causal=True)
    moved = 0.0
    for h in range(2):
        for i in range(n):
            m = np.max(scale * k[0, h, :i + 1] @ q[0, h, i])
            ref = _wls_intercept(q[0, h, i], k[0, h, :i + 1], v[0, h, :i + 1], scale, lam * np.exp(m))
            np.testing.assert_allclose(out[0, h, i], ref, rtol=1e-8, atol=1e-10)
            moved = max(moved, np.abs(out[0, h, i] - plain[0, h, i]).max())
    assert moved > 1e-3            # the two variants are different functions at these scores
    # ... and the same thing through the per-token input of the definition mode
    m_all = np.array([[[np.max(scale * k[0, h, :i + 1] @ q[0, h, i]) for i in range(n)] for h in range(2)]])
    np.testing.assert_allclose(out, oracle.forward(q, k, v, scale, lam * np.exp(m_all)), rtol=1e-10, atol=1e-12)


def test_decode_ridge_variants_equal_last_prefill_row(oracle):
    rng = np.random.default_rng(24)
    B, H, Lmax, d, dv = 2, 3, 12, 3, 4
    kc = rng.standard_normal((B, H, Lmax, d))
    vc = rng.standard_normal((B, H, Lmax, dv))
    qd = rng.standard_normal((B, H, d))
    lens = np.array([12, 5], dtype=np.int32)
    lam = rng.uniform(1e-2, 0.3, size=(B, H))
    for mode in ("definition", "printed"):
        out = oracle.decode(qd, kc, vc, lens, 0.8, lam, ridge_mode=mode)
        for b in range(B):
            L = int(lens[b])
            qfull = np.zeros((1, H, L, d))
            qfull[0, :, L - 1] = qd[b]
            lam_rows = np.repeat(lam[b][None, :, None], L, axis=2)
            ref = oracle.forward(qfull, kc[b:b + 1, :, :L], vc[b:b + 1, :, :L], 0.8, lam_rows, ridge_mode=mode)
            np.testing.assert_allclose(out[b], ref[0, :, L - 1], rtol=1e-12, atol=1e-14)
