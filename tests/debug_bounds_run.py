"""Run in a process of its own with LLA_LIBRARY pointing at the bounds-checking debug build (liblla_debug.so):
small forward, decode and backward calls that reach every kernel family, each with a status array.  Prints one
JSON object: per call its name, the status words and the largest row error against the oracle.  The test that
spawns this checks that no store was out of range (LLA_STATUS_BOUNDS == 0) and that parity holds as in the product
build.  Not collected by pytest (no test functions)."""
import json
import sys
from pathlib import Path

import numpy as np
import torch

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))

from oracle import lla_backward_oracle, lla_oracle  # noqa: E402
from paper_2510_01450_b200 import binding as L  # noqa: E402
from paper_2510_01450_b200 import inputs  # noqa: E402
from tests.gpu_util import LLA_DT, dev, row_err, stream_ptr  # noqa: E402


def status_array():
    return torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")


def forward_case(name, w, **kw):
    q, k, v = inputs.make_prefill(w)
    ref = lla_oracle.forward(q, k, v, w.scale, w.lam)
    dq, dk, dv_ = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    out = torch.full((w.B, w.H, w.n, w.dv), float("nan"), dtype=torch.float32, device="cuda")
    st = status_array()
    nbytes = L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, LLA_DT[w.dtype], L.LLA_IMPL_AUTO)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    L.lla_forward_ex(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, in_dtype=LLA_DT[w.dtype],
                     out_dtype=L.LLA_F32, device_status=st, workspace=ws if nbytes else None, workspace_bytes=nbytes,
                     stream=stream_ptr(), **kw)
    torch.cuda.synchronize()
    return {"name": name, "status": st.cpu().tolist(), "err": float(row_err(out.cpu().numpy(), ref).max())}


def decode_case(name, w, splits):
    q, kc, vc, lens = inputs.make_decode(w)
    ref = lla_oracle.decode(q, kc, vc, lens, w.scale, w.lam)
    dq, dk, dv_ = dev(q, "bf16"), dev(kc, "bf16"), dev(vc, "bf16")
    dl = torch.from_numpy(lens).cuda()
    out = torch.full((w.B, w.H, w.dv), float("nan"), dtype=torch.float32, device="cuda")
    st = status_array()
    nbytes = L.lla_decode_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, splits)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    L.lla_decode_ex(dq, dk, dv_, dl, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, out_dtype=L.LLA_F32, splits=splits,
                    device_status=st, workspace=ws, workspace_bytes=nbytes, stream=stream_ptr())
    torch.cuda.synchronize()
    return {"name": name, "status": st.cpu().tolist(), "err": float(row_err(out.cpu().numpy(), ref).max())}


def backward_case(name, w):
    q, k, v = inputs.make_prefill(w)
    g = inputs.make_upstream_grad(w)
    ref = lla_backward_oracle.backward(q, k, v, g, w.scale, w.lam)
    dq, dk, dv_, dg = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16"), dev(g, "f32")
    shape = (w.B, w.H, w.n, w.d)
    out, rho = (torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(2))
    stats = torch.empty((w.B, w.H, w.n, 3), dtype=torch.float32, device="cuda")
    L.lla_forward_ex(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.d, w.scale, w.lam, out_dtype=L.LLA_F32, rho=rho, stats=stats,
                     stream=stream_ptr())
    grads = [torch.full(shape, float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    nbytes = L.lla_backward_workspace_bytes(w.B, w.H, w.n, w.d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    st = status_array()
    L.lla_backward_ex(dq, dk, dv_, out, dg, rho, stats, *grads, w.B, w.H, w.n, w.d, w.scale, w.lam, device_status=st,
                      workspace=ws, workspace_bytes=nbytes, stream=stream_ptr())
    torch.cuda.synchronize()
    err = 0.0
    for a, b in zip(grads, ref):
        a = a.cpu().numpy().astype(np.float64)
        rn = np.linalg.norm(b.reshape(-1, w.d), axis=1)
        diff = np.linalg.norm((a - b).reshape(-1, w.d), axis=1)
        err = max(err, float((diff / np.maximum(rn, 0.1 * np.median(rn))).max()))
    return {"name": name, "status": st.cpu().tolist(), "err": err}


def main():
    c2, c5 = inputs.CONFIGS[2], inputs.CONFIGS[5]
    cases = [
        forward_case("forward d64 ragged", c2.shrink(B=1, H=2, n=333, seed=400)),
        forward_case("forward d128", c2.shrink(B=1, H=2, n=300, d=128, dv=128, seed=401)),
        forward_case("forward d64 several tiles", c2.shrink(B=2, H=1, n=700, seed=402)),
        forward_case("forward fp32 d16", inputs.CONFIGS[1].shrink(B=1, H=2, n=200, seed=403)),
        decode_case("decode split", c5.shrink(B=3, H=2, n=1500, len_min=40, len_max=1500, seed=404), 3),
        decode_case("decode unsplit", c5.shrink(B=2, H=2, n=700, len_min=200, len_max=700, seed=405), 1),
        backward_case("backward d64", c2.shrink(B=1, H=2, n=333, seed=406)),
        backward_case("backward d128", c2.shrink(B=1, H=1, n=300, d=128, dv=128, seed=407)),
    ]
    print(json.dumps({"library": str(L._LIB_PATH), "cases": cases}))


if __name__ == "__main__":
    main()
