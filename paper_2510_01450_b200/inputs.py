"""Seeded synthetic inputs for the five LLA workloads.

This module holds no attention arithmetic: it only draws random tensors with the
shapes, value distributions and structure of the workloads and rounds them once
to the I/O dtype.  Both the CUDA tests/bench and the CPU oracle's tests use it,
so the two sides see bit-identical inputs.

All arrays are returned as numpy float32.  For the bf16 workloads every value is
already rounded to the nearest bf16 (ties to even), so converting to a bf16
tensor afterwards is exact and the float32 copy handed to the oracle is the very
same number.

Workloads (the paper benchmarks "a range of dimensions and batch sizes" without
listing them; these five stand in for them):
  1  fp32, B=1,H=1,n=256,d=dv=16, q,k,v ~ N(0,1)/sqrt(d), lambda=1e-2, seed 0
  2  bf16, B=4,H=8,n=1024,d=dv=64, q,k ~ N(0,1/d), v ~ N(0,1), lambda=1e-3
  3  bf16, B=2,H=16,n=4096,d=dv=64, test-time-regression shape (Section 4.1):
     keys N(0,I/d), v_j = A_s k_j + 0.1*noise with A_s ~ N(0,1/d) redrawn every
     512 tokens, query i = key i+1, lambda=1e-2
  4  bf16, B=1,H=16,n=16384,d=dv=128, q,k ~ N(0,1/d), v ~ N(0,1), lambda=1e-3
  5  bf16 decode, 64 sequences, H=16, d=dv=64, cache lengths uniform in
     [1024, 8192], q,k ~ N(0,1/d), v ~ N(0,1), lambda=1e-3
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str          # "prefill" or "decode"
    dtype: str         # "f32" or "bf16"
    B: int
    H: int
    n: int             # prefill: sequence length; decode: Lmax of the cache
    d: int
    dv: int
    lam: float
    seed: int
    recipe: str        # "iid" or "regression"
    len_min: int = 0   # decode only
    len_max: int = 0
    segment: int = 512  # regression recipe: tokens per linear map

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d))

    def shrink(self, **kw) -> "Workload":
        """Same recipe at other sizes (used by tests that need the oracle to finish fast)."""
        return replace(self, **kw)


CONFIGS = {
    1: Workload("cfg1_f32_n256_d16", "prefill", "f32", 1, 1, 256, 16, 16, 1e-2, 0, "iid"),
    2: Workload("cfg2_bf16_n1024_d64", "prefill", "bf16", 4, 8, 1024, 64, 64, 1e-3, 2, "iid"),
    3: Workload("cfg3_bf16_regression_n4096_d64", "prefill", "bf16", 2, 16, 4096, 64, 64, 1e-2, 3,
                "regression"),
    4: Workload("cfg4_bf16_n16384_d128", "prefill", "bf16", 1, 16, 16384, 128, 128, 1e-3, 4, "iid"),
    5: Workload("cfg5_bf16_decode_b64_h16_d64", "decode", "bf16", 64, 16, 8192, 64, 64, 1e-3, 5,
                "iid", len_min=1024, len_max=8192),
}


def _finish(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_to_bf16(x) if dtype == "bf16" else x


def make_prefill(w: Workload):
    """Return (q, k, v) float32 arrays of shape [B,H,n,d], [B,H,n,d], [B,H,n,dv]."""
    assert w.kind == "prefill"
    rng = np.random.default_rng(w.seed)
    B, H, n, d, dv = w.B, w.H, w.n, w.d, w.dv
    inv = np.float32(1.0 / np.sqrt(d))
    if w.recipe == "iid":
        q = rng.standard_normal((B, H, n, d), dtype=np.float32) * inv
        k = rng.standard_normal((B, H, n, d), dtype=np.float32) * inv
        v = rng.standard_normal((B, H, n, dv), dtype=np.float32)
        if w.name.startswith("cfg1"):
            v = v * np.float32(1.0 / np.sqrt(d))   # the fp32 n = 256, d = 16 case scales q, k and v alike
    elif w.recipe == "regression":
        keys, A, noise = _regression_draws(w, rng)
        k = keys[:, :, :n]
        q = keys[:, :, 1:]                        # the query at position i is the next key
        v = np.empty((B, H, n, dv), dtype=np.float32)
        for s in range(A.shape[2]):
            lo, hi = s * w.segment, min(n, (s + 1) * w.segment)
            v[:, :, lo:hi] = np.einsum("bhvd,bhjd->bhjv", A[:, :, s], k[:, :, lo:hi]) \
                + np.float32(REGRESSION_NOISE) * noise[:, :, lo:hi]
    else:
        raise ValueError(w.recipe)
    return _finish(q, w.dtype), _finish(k, w.dtype), _finish(v, w.dtype)


REGRESSION_NOISE = 0.1     # standard deviation of the value noise of the regression recipe


def _regression_draws(w: Workload, rng):
    """The regression recipe's random draws, in the order make_prefill consumes them: n + 1 keys, one linear map
    per segment, the value noise."""
    B, H, n, d, dv = w.B, w.H, w.n, w.d, w.dv
    inv = np.float32(1.0 / np.sqrt(d))
    keys = rng.standard_normal((B, H, n + 1, d), dtype=np.float32) * inv
    nseg = (n + w.segment - 1) // w.segment
    A = rng.standard_normal((B, H, nseg, dv, d), dtype=np.float32) * inv
    noise = rng.standard_normal((B, H, n, dv), dtype=np.float32)
    return keys, A, noise


def regression_targets(w: Workload) -> np.ndarray:
    """For the regression recipe: the noise-free value of the query at every position, A_s q_i with s the segment
    of the NEXT position (query i is key i + 1), [B,H,n,dv] float32.  A regressor that has identified the
    current segment's linear map predicts exactly this; at a segment's last position the query already belongs to
    the next segment, whose map nothing seen so far determines."""
    assert w.recipe == "regression"
    keys, A, _ = _regression_draws(w, np.random.default_rng(w.seed))
    n = w.n
    out = np.empty((w.B, w.H, n, w.dv), dtype=np.float32)
    nseg = A.shape[2]
    for s in range(nseg + 1):
        lo, hi = max(0, s * w.segment - 1), min(n, (s + 1) * w.segment - 1)     # positions whose next position lies in s
        if lo >= hi:
            continue
        a_s = A[:, :, min(s, nseg - 1)]
        out[:, :, lo:hi] = np.einsum("bhvd,bhjd->bhjv", a_s, keys[:, :, lo + 1:hi + 1])
    return out


def make_upstream_grad(w: Workload, dtype: str = "f32") -> np.ndarray:
    """Upstream gradient g = dL/d(out) for the backward pass, [B,H,n,dv]: standard normal entries (the
    gradient a unit-variance loss head hands back), drawn from a stream of its own so that q, k, v
    of the same workload are unchanged."""
    rng = np.random.default_rng([w.seed, 0x6772])
    return _finish(rng.standard_normal((w.B, w.H, w.n, w.dv), dtype=np.float32), dtype)


def make_decode(w: Workload):
    """Return (q [B,H,d], kcache [B,H,Lmax,d], vcache [B,H,Lmax,dv], lens [B] int32)."""
    assert w.kind == "decode"
    rng = np.random.default_rng(w.seed)
    B, H, Lmax, d, dv = w.B, w.H, w.n, w.d, w.dv
    inv = np.float32(1.0 / np.sqrt(d))
    lens = rng.integers(w.len_min, w.len_max + 1, size=B).astype(np.int32)
    q = rng.standard_normal((B, H, d), dtype=np.float32) * inv
    kc = rng.standard_normal((B, H, Lmax, d), dtype=np.float32)
    kc *= inv
    vc = rng.standard_normal((B, H, Lmax, dv), dtype=np.float32)
    return _finish(q, w.dtype), _finish(kc, w.dtype), _finish(vc, w.dtype), lens


def sample_rows(w: Workload, per_head: int, heads: int, seed: int = 0, dense_below: int = 0,
                tile: int = 128) -> np.ndarray:
    """Flat row indices (b*H+h)*n+i for sampled parity checks on large workloads.

    For ``heads`` (b,h) pairs spread over the batch: every row below ``dense_below``, every row
    of the last ``tile`` rows, and ``per_head`` rows drawn uniformly from the rest.
    """
    rng = np.random.default_rng(seed + 1000)
    BH = w.B * w.H
    bhs = np.unique(np.linspace(0, BH - 1, num=min(heads, BH)).round().astype(np.int64))
    out = []
    for bh in bhs:
        fixed = np.concatenate([np.arange(0, min(dense_below, w.n)),
                                np.arange(max(0, w.n - tile), w.n)])
        rnd = rng.integers(0, w.n, size=per_head)
        out.append(bh * w.n + np.unique(np.concatenate([fixed, rnd])))
    return np.concatenate(out).astype(np.int64)


def shard_units(n_units: int, rank: int, world: int):
    """Contiguous split of independent (batch, head) units across ranks: [lo, hi) for ``rank``.

    The (b,h) problems are independent (the paper's multi-head extension), so the path shards
    with no exchange step.
    """
    base, rem = divmod(n_units, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
