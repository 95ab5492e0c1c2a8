"""Helpers shared by the GPU tests: tensor conversion and the parity metric."""
import numpy as np
import torch

from paper_2510_01450_b200 import binding as L

TORCH_DT = {"bf16": torch.bfloat16, "f32": torch.float32}
LLA_DT = {"bf16": L.LLA_BF16, "f32": L.LLA_F32}


def dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 numpy (already rounded to the I/O dtype) -> contiguous CUDA tensor of that dtype (exact)."""
    return torch.from_numpy(np.ascontiguousarray(x)).to(TORCH_DT[dtype]).cuda().contiguous()


def stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


def row_err(got, ref) -> np.ndarray:
    """Row-wise relative L2 error |o_i - ref_i| / |ref_i| over the last axis (the gating metric)."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, ref.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    return np.linalg.norm(got - ref, axis=1) / np.linalg.norm(ref, axis=1)


def elem_err(got, ref) -> np.ndarray:
    """Element-wise error scaled by the row's largest entry, max_c |o_ic - ref_ic| / max_c |ref_ic| (a second
    gate beside the row norm: one bad element of an otherwise exact row shows here undiluted)."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, ref.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    return np.abs(got - ref).max(axis=1) / np.abs(ref).max(axis=1)


def forward(w, q, k, v, out_dtype=None, causal=True, **kw):
    """Run lla_forward_ex on a workload's arrays; returns the output as float64 numpy [B,H,n,dv]."""
    out_dtype = out_dtype or w.dtype
    dq, dk, dv_ = dev(q, w.dtype), dev(k, w.dtype), dev(v, w.dtype)
    out = torch.full((w.B, w.H, w.n, w.dv), float("nan"), dtype=TORCH_DT[out_dtype], device="cuda")
    if "workspace" not in kw:
        # the optional scratch a caller would normally provide (lla_forward takes it from the memory pool)
        nbytes = L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.dv, LLA_DT[w.dtype], kw.get("impl", L.LLA_IMPL_AUTO))
        if nbytes:
            kw["workspace"] = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            kw["workspace_bytes"] = nbytes
    L.lla_forward_ex(dq, dk, dv_, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, causal=causal,
                     in_dtype=LLA_DT[w.dtype], out_dtype=LLA_DT[out_dtype], stream=stream_ptr(), **kw)
    torch.cuda.synchronize()
    return out.float().cpu().numpy().astype(np.float64)
