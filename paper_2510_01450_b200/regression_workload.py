"""Test-time regression with the LLA forward pass (Section 4.1 of the paper, the experiment behind its
regression-fit figure, in a reduced form).

Keys are Gaussian, values follow a linear map of the keys that is redrawn every ``segment`` tokens
(non-stationary data), plus noise; the query at position i is the next key, and the quantity of interest
is how well the attention output at position i predicts the next value.  The module runs the CUDA forward
twice on the same inputs -- with the workload's ridge (local linear regression) and with a very large ridge,
which turns the same kernel into softmax attention, the local-constant (Nadaraya-Watson) limit of Section
2.2 -- and reports the position-wise mean squared error of both against the noise-free next value, in units
of the noise variance.  The comparison systems of the paper's figure (linear attention, MesaNet) and its
cone-segment key generator are not part of it.

    python -m paper_2510_01450_b200.regression_workload [--d 16,64,128] [--segments 128,512,2048] [--n 4096]

prints one JSON line per (d, segment) case.  ``run_case`` is what the tests call.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as L
from . import inputs

SOFTMAX_RIDGE = 1e7        # ridge at which the LLA output has converged to softmax attention (error ~ 1 / ridge)


def _forward(torch, w, dq, dk, dv, lam):
    out = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.float32, device="cuda")
    nbytes = L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.dv)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    L.lla_forward_ex(dq, dk, dv, out, w.B, w.H, w.n, w.d, w.dv, w.scale, lam, causal=1, out_dtype=L.LLA_F32,
                     workspace=ws if nbytes else None, workspace_bytes=nbytes,
                     stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def run_case(d: int, segment: int, n: int = 4096, B: int = 2, H: int = 4, lam: float = 1e-2, seed: int = 3):
    """One case: returns a dict with the workload, the two outputs' position-wise MSE (mean over batch, head and
    value dimension, divided by the noise variance) as arrays ``mse_lla`` and ``mse_softmax`` of length n, the
    outputs themselves (``out_lla``, ``out_softmax``, float32 [B,H,n,dv]) and the inputs (for an oracle check)."""
    import torch
    w = inputs.CONFIGS[3].shrink(B=B, H=H, n=n, d=d, dv=d, lam=lam, seed=seed, segment=segment,
                                 name=f"regression_n{n}_d{d}_seg{segment}")
    q, k, v = inputs.make_prefill(w)
    target = inputs.regression_targets(w).astype(np.float64)
    dq, dk, dv = (torch.from_numpy(x).to(torch.bfloat16).cuda() for x in (q, k, v))
    out_lla = _forward(torch, w, dq, dk, dv, lam)
    out_soft = _forward(torch, w, dq, dk, dv, SOFTMAX_RIDGE)
    noise_var = inputs.REGRESSION_NOISE ** 2
    mse = lambda o: ((o.astype(np.float64) - target) ** 2).mean(axis=(0, 1, 3)) / noise_var     # noqa: E731
    return {"workload": w, "inputs": (q, k, v), "out_lla": out_lla, "out_softmax": out_soft,
            "mse_lla": mse(out_lla), "mse_softmax": mse(out_soft)}


def summarise(case) -> dict:
    """Bucket the position-wise errors by how many keys of the current linear map a position has seen: fewer than
    d + 1 (no linear fit is determined), up to 2d + 2, up to 4d, and the rest of the segment; separately for the
    first segment (stationary data) and for the later ones (keys of earlier maps are still visible)."""
    w = case["workload"]
    d, seg, n = w.d, w.segment, w.n
    pos = np.arange(n)
    in_seg = (pos + 1) % seg            # keys of the next position's map that position i can see
    seg_of_next = (pos + 1) // seg
    valid = in_seg > 0                  # at a segment's last position the query belongs to an unseen map
    edges = [1, d + 2, 2 * d + 3, 4 * d + 1, seg]
    names = ["seen<=d+1", "d+1<seen<=2d+2", "2d+2<seen<=4d", "seen>4d"]
    rows = {}
    for part, sel in (("first_segment", seg_of_next == 0), ("later_segments", seg_of_next > 0)):
        rows[part] = {}
        for name, lo, hi in zip(names, edges[:-1], edges[1:]):
            m = valid & sel & (in_seg >= lo) & (in_seg < hi)
            if m.any():
                rows[part][name] = {"positions": int(m.sum()), "mse_lla": float(case["mse_lla"][m].mean()),
                                    "mse_softmax": float(case["mse_softmax"][m].mean())}
    return {"workload": w.name, "B": w.B, "H": w.H, "n": n, "d": d, "segment": seg, "lambda": w.lam,
            "softmax_ridge": SOFTMAX_RIDGE, "unit": "mean squared error / noise variance", "buckets": rows}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", default="16,64,128")
    ap.add_argument("--segments", default="128,512,2048")
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--heads", type=int, default=4)
    args = ap.parse_args()
    for d in (int(x) for x in args.d.split(",")):
        for seg in (int(x) for x in args.segments.split(",")):
            print(json.dumps(summarise(run_case(d, seg, n=args.n, H=args.heads))), flush=True)


if __name__ == "__main__":
    main()
