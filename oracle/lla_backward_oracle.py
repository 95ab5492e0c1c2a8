"""Float64 CPU oracle for the gradient of the causal LLA forward pass.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
bench's CPU-baseline leg.  The CUDA library never imports this module and this
module never imports the CUDA package.

What it computes.  The forward pass maps (Q, K, V) to the local-linear
intercepts o_i (paper Section 2.3, Eq. "query_specific" and Eq. "lla").  For an
upstream gradient g_i = dL/do_i (the paper's g_i of the backward appendix) the
backward pass returns dL/dQ, dL/dK, dL/dV.  The gradient has a plain
definition -- the derivative of the forward map -- so the oracle is that
definition written out: the forward is evaluated from its defining formulas
(explicit z_ij = k_j - q_i, explicit moments omega_i, mu_i, Sigma_i, a dense
solve) in float64 with plain PyTorch CPU ops, and reverse-mode differentiation
of exactly those ops gives the gradient.  None of the hand-derived expressions
of the backward appendix (u_i, Delta_mu, relmm terms) is used here, so the
oracle is independent of them; ``tests/test_backward_oracle_pins.py`` pins it
against finite differences of the separate C forward oracle, closed forms and
the appendix's own formulas.

Weights are exp(score - m_i) with the ridge lambda * exp(-m_i): the forward
value does not depend on the shift m_i (the joint scaling of weights and ridge
leaves Eq. "lla" unchanged), so m_i is treated as a constant and carries no
gradient.
"""
from __future__ import annotations

import numpy as np
import torch


def _forward_rows(Q, K, V, rows, scale, lam, causal, window=0, visible=None, q_offset=0):
    """o_i for the given row indices of one head, from the definition (float64 tensors).  window > 0 (causal only):
    row i sees its last `window` positions, keys max(0, i - window + 1) .. i (the sliding window that the paper's
    discussion section suggests; the sums of Eq. "query_specific" then run over those keys).  visible (optional, bool
    [n, n]): row i sees key j only where visible[i, j] as well (sparse attention: the same sums over fewer keys).
    q_offset: Q holds only the queries of positions q_offset .. n - 1 (a chunk of queries against a longer key
    sequence); `rows` are positions."""
    n = K.shape[0]
    d = K.shape[1]
    L = int(rows.max()) + 1 if causal else n
    Kl, Vl = K[:L], V[:L]
    Qr = Q[rows - q_offset]
    s = scale * (Qr @ Kl.T)                                        # scores, Section 3.1
    if causal:
        mask = torch.arange(L)[None, :] <= rows[:, None]           # row i sees keys j <= i
        if window > 0:
            mask = mask & (torch.arange(L)[None, :] > rows[:, None] - window)
    else:
        mask = torch.ones(len(rows), L, dtype=torch.bool)
    if visible is not None:
        mask = mask & torch.as_tensor(np.asarray(visible)[rows.numpy()][:, :L])
    m = torch.where(mask, s, torch.full_like(s, -torch.inf)).max(dim=1).values.detach()
    w = torch.where(mask, torch.exp(s - m[:, None]), torch.zeros_like(s))
    lam_i = (lam[rows] if torch.is_tensor(lam) else lam) * torch.exp(-m)    # one ridge per row when lam is a tensor
    Z = Kl[None, :, :] - Qr[:, None, :]                            # z_ij = k_j - q_i
    mu = torch.einsum("rj,rjc->rc", w, Z)                          # mu_i
    Sigma = torch.einsum("rj,rjc,rje->rce", w, Z, Z) + lam_i[:, None, None] * torch.eye(d, dtype=Q.dtype)
    rho = torch.linalg.solve(Sigma, mu)                            # Sigma_i rho_i = mu_i
    c = w * (1.0 - torch.einsum("rjc,rc->rj", Z, rho))             # w_ij (1 - z_ij^T rho_i)
    return (c @ Vl) / c.sum(dim=1, keepdim=True)                   # Eq. "lla"


def backward(q, k, v, g, scale, lam, causal=True, chunk=32, want_dlambda=False, window=0, visible=None):
    """Gradients of sum_i <g_i, o_i> with respect to q, k, v.

    k: [B, H, n, d]; v: [B, H, n, dv]; q: [B, H, nq, d] and g: [B, H, nq, dv] with nq <= n: the queries (and their
    upstream gradients) of the last nq positions, a chunk of queries against a longer key sequence; nq = n is the
    whole sequence.  numpy arrays (any float dtype; widened to float64).
    visible: optional bool [n, n] or [B * H, n, n] (row, key) visibility on top of causality (see _forward_rows).
    Returns (dq, dk, dv) as float64 numpy arrays of the inputs' shapes; with want_dlambda also
    dlambda [B, H, n], the derivative with respect to a ridge of its own per query row (the paper's
    learnable per-token regularisation, Appendix on the regularisation), each evaluated at lam.
    """
    q, k, v, g = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g))
    B, H, nq, _ = q.shape
    n = k.shape[2]
    off = n - nq              # the queries are the last nq positions (causal); nq = n is the whole sequence
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dlam = np.zeros((B, H, nq))
    for b in range(B):
        for h in range(H):
            Q = torch.tensor(q[b, h], requires_grad=True)
            K = torch.tensor(k[b, h], requires_grad=True)
            V = torch.tensor(v[b, h], requires_grad=True)
            G = torch.tensor(g[b, h])
            lam_rows = torch.full((n,), float(lam), dtype=torch.float64, requires_grad=True)
            for r0 in range(off, n, chunk):
                rows = torch.arange(r0, min(n, r0 + chunk))
                vis = None if visible is None else (visible if np.ndim(visible) == 2 else visible[b * H + h])
                o = _forward_rows(Q, K, V, rows, float(scale), lam_rows if want_dlambda else float(lam), bool(causal),
                                  int(window), vis, off)
                (o * G[rows - off]).sum().backward()
            dq[b, h], dk[b, h], dv[b, h] = Q.grad.numpy(), K.grad.numpy(), V.grad.numpy()
            if want_dlambda:
                dlam[b, h] = lam_rows.grad.numpy()[off:]
    return (dq, dk, dv, dlam) if want_dlambda else (dq, dk, dv)


def backward_rows(q, k, v, g, scale, lam, rows, window=0):
    """The share of the gradient that the given query rows of ONE head contribute (causal): q, k [n, d]; v, g [n, dv];
    rows a sequence of row indices.  Returns (dq_rows [len(rows), d], dk [n, d], dv [n, dv]) for the loss
    sum_{i in rows} <g_i, o_i>: dq_rows are the full gradient's rows (a query enters its own row only), dk and dv its
    shares from these rows -- complete for every key that no other row sees, e.g. the last m keys when rows are the
    last m rows.  Same definition and operations as backward(), one row at a time (sizes the full-size tests need)."""
    q, k, v, g = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g))
    Q = torch.tensor(q, requires_grad=True)
    K = torch.tensor(k, requires_grad=True)
    V = torch.tensor(v, requires_grad=True)
    G = torch.tensor(g)
    for i in rows:
        r = torch.tensor([int(i)])
        o = _forward_rows(Q, K, V, r, float(scale), float(lam), True, int(window))
        (o * G[r]).sum().backward()
    return Q.grad.numpy()[np.asarray(list(rows), dtype=np.int64)], K.grad.numpy(), V.grad.numpy()


def forward(q, k, v, scale, lam, causal=True, chunk=32, window=0, visible=None):
    """The forward values the gradient above differentiates (used by the pins to tie this module's
    forward to the C oracle's)."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    B, H, n, _ = q.shape
    out = np.zeros(v.shape[:2] + (n, v.shape[3]))
    with torch.no_grad():
        for b in range(B):
            for h in range(H):
                Q, K, V = (torch.tensor(a[b, h]) for a in (q, k, v))
                for r0 in range(0, n, chunk):
                    rows = torch.arange(r0, min(n, r0 + chunk))
                    vis = None if visible is None else (visible if np.ndim(visible) == 2 else visible[b * H + h])
                    out[b, h, r0:r0 + len(rows)] = _forward_rows(Q, K, V, rows, float(scale), float(lam),
                                                                 bool(causal), int(window), vis).numpy()
    return out
