#!/usr/bin/env python
"""Benchmark of the LLA hot path on B200.  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 2|3|4]

Headline: the causal forward (prefill) on the largest single-GPU prefill workload, bf16 B=1, H=16,
n=16384, d=dv=128.  A step is one pass of the whole forward path (direct early rows + iterative rows)
over one batch.  The line also carries the two smaller prefill workloads (n=1024 and n=4096, d=64)
as legs measured the same way, the decode step against HBM bandwidth, the backward pass, the
end-to-end host-buffer number and the CPU oracle baseline with parity figures per leg.  With N > 1
every rank runs the whole batch on its own GPU (independent (batch, head) problems, no collective
on the data path: weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_01450_b200 import inputs  # noqa: E402

METRIC = "lla_prefill_tokens_per_s"
UNIT = "tokens/s"
HEADLINE = 4          # the largest single-GPU prefill workload
LEGS = (2, 3)         # the other bf16 prefill workloads, reported as sub-objects
L2_BYTES = 126e6
# DRAM bytes (read + write) per launch of the dominant kernel from the ncu captures summarised under
# profiles/: (bytes, summary file).  Workload 4 was captured with 2 of its 16 heads and scaled by 8
# (traffic is per head: Q, K, V once).
NCU_TRAFFIC = {
    2: (12.68e6, "profiles/forward_tc_kernel_cfg2.md"),
    3: (4 * 17.06e6, "profiles/forward_tc_kernel_cfg3.md (8 of 32 units captured, x 4)"),
    4: (8 * (33.67e6 + 2.58e6), "profiles/forward_tc_kernel_cfg4.md (2 of 16 heads captured, x 8)"),
}
NCU_DECODE_TRAFFIC = (1.188e9 + 24.2e6 + 34.3e6, "profiles/decode_tc_kernel_cfg5.md")   # streaming read + record write, solve read


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML while a timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
        self.period = period_s

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def merge_clocks(parts):
    """One clocks object for the whole run from the per-region samplers."""
    samples = [s for p in parts for s in p.samples]
    reasons = sorted(set().union(*[p.reasons for p in parts])) if parts else []
    mx = next((p.max_mhz for p in parts if p.max_mhz), None)
    return {"sm_mhz": float(np.median(samples)) if samples else None, "sm_max_mhz": mx, "reasons": reasons,
            "samples": len(samples)}


def algorithmic_flops(w, iters: np.ndarray, iterative_only: bool = False) -> float:
    """N_p (8d + 2dv) + 6d sum_i (i+1) T_i per head, with the CG iterations actually executed
    (rows solved directly contribute no iteration term; with iterative_only they are left out)."""
    n, d, dv = w.n, w.d, w.dv
    it = iters.reshape(-1, n).astype(np.float64)
    vis = np.arange(1, n + 1, dtype=np.float64)
    base = (it >= 0) if iterative_only else np.ones_like(it, dtype=bool)
    return float((8 * d + 2 * dv) * (base * vis).sum() + 6.0 * d * (np.maximum(it, 0.0) * vis).sum())


def workload_config(w):
    """The keys both arms print: the workload and how L2 is kept out of the measurement."""
    set_bytes = 4 * w.B * w.H * w.n * w.d * 2
    rot = rotate_sets(w)
    return {"workload": w.name, "B": w.B, "H": w.H, "n": w.n, "d": w.d, "dv": w.dv, "lambda": w.lam, "causal": True,
            "l2": f"inputs rotate over {rot} sets of {set_bytes / 1e6:.0f} MB ({rot * set_bytes / 1e6:.0f} MB > 126 MB L2)"}


def rotate_sets(w) -> int:
    """Input sets cycled through so that no step finds its inputs in L2 (at least 2, together > 2 x L2)."""
    set_bytes = 4 * w.B * w.H * w.n * w.d * 2
    return int(max(2, min(16, np.ceil(2.2 * L2_BYTES / set_bytes))))


def oracle_sample_rows(w, n_rows: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return np.sort(rng.choice(w.B * w.H * w.n, size=min(n_rows, w.B * w.H * w.n), replace=False)).astype(np.int64)


def run_reference(args):
    """Reference arm: the float64 CPU oracle, as it stands, on a bounded sample of the workload."""
    rank = env_int("RANK", 0)
    if rank != 0:
        return
    from oracle import lla_oracle
    w = inputs.CONFIGS[args.workload]
    q, k, v = inputs.make_prefill(w)
    total_rows = w.B * w.H * w.n
    # calibrate: rows are drawn uniformly over (batch, head, position), so the sample's mean cost
    # per row equals the workload's
    probe = oracle_sample_rows(w, 128, 1)
    t0 = time.perf_counter()
    lla_oracle.forward_rows(q, k, v, w.scale, w.lam, rows=probe)
    per_row = (time.perf_counter() - t0) / probe.size
    budget_s = 120.0
    rows_per_step = int(max(32, min(total_rows, budget_s / max(per_row, 1e-9) / (args.steps + args.warmup))))
    for i in range(args.warmup):
        lla_oracle.forward_rows(q, k, v, w.scale, w.lam, rows=oracle_sample_rows(w, rows_per_step, 100 + i))
    t0 = time.perf_counter()
    for i in range(args.steps):
        lla_oracle.forward_rows(q, k, v, w.scale, w.lam, rows=oracle_sample_rows(w, rows_per_step, 200 + i))
    dt = time.perf_counter() - t0
    value = rows_per_step / w.H * args.steps / dt      # a token is one position with all H heads
    sample = (f"{rows_per_step} of {total_rows} (head, position) rows per step, drawn uniformly over "
              "(batch, head, position); tokens = rows / H")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": lla_oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


class Prefill:
    """One prefill workload resident on the device: rotating input sets, outputs, timing helpers."""

    def __init__(self, L, torch, w, local):
        self.L, self.torch, self.w, self.local = L, torch, w, local
        self.stream = torch.cuda.current_stream()
        self.sp = self.stream.cuda_stream
        self.host = inputs.make_prefill(w)
        hq, hk, hv = (torch.from_numpy(x).to(torch.bfloat16) for x in self.host)
        self.host_bf16 = (hq, hk, hv)
        self.rot = rotate_sets(w)
        self.sets = []
        for r in range(self.rot):
            # every set is the same seeded batch with its (batch, head) order rotated: same work, new addresses
            sh = r % (w.B * w.H)
            self.sets.append(tuple(torch.roll(t.reshape(w.B * w.H, w.n, -1), sh, 0).reshape(t.shape).contiguous().cuda()
                                   for t in (hq, hk, hv)))
        self.outs = [torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.bfloat16, device="cuda") for _ in range(self.rot)]
        self.set_bytes = sum(t.numel() * t.element_size() for t in self.sets[0]) + self.outs[0].numel() * 2
        nws = L.lla_forward_workspace_bytes(w.B, w.H, w.n, w.d, w.dv)
        self.ws = torch.empty(max(nws, 256), dtype=torch.uint8, device="cuda") if nws else None
        self.ws_bytes = nws
        self.precondition = 0

    def step(self, i, phases=0):
        w, L = self.w, self.L
        q, k, v = self.sets[i % self.rot]
        L.lla_forward_ex(q, k, v, self.outs[i % self.rot], w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, causal=1,
                         phases=phases, workspace=self.ws, workspace_bytes=self.ws_bytes, stream=self.sp,
                         cg_precondition=self.precondition)

    def probe(self):
        """Iterations actually executed (for the algorithmic flop count) and an fp32 copy of set 0's
        output for the parity figures; outside every timed region."""
        w, L, torch = self.w, self.L, self.torch
        iters = torch.zeros((w.B, w.H, w.n), dtype=torch.int32, device="cuda")
        status = torch.zeros(L.LLA_STATUS_WORDS, dtype=torch.int32, device="cuda")
        out32 = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.float32, device="cuda")
        L.lla_forward_ex(*self.sets[0], out32, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, causal=1, iters=iters,
                         out_dtype=L.LLA_F32, device_status=status, workspace=self.ws, workspace_bytes=self.ws_bytes,
                         stream=self.sp)
        torch.cuda.synchronize()
        self.iters = iters.cpu().numpy()
        self.status = status.cpu().numpy()
        self.out32 = out32.cpu().numpy().reshape(-1, w.dv)
        del out32

    def timed(self, steps, warmup, phases=0, barrier=None):
        """(ms for `steps` launches, clock summary): CUDA events on the launching stream."""
        torch = self.torch
        for i in range(warmup):
            self.step(i, phases)
        (barrier or torch.cuda.synchronize)()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(self.local) as clk:
            e0.record(self.stream)
            for i in range(steps):
                self.step(warmup + i, phases)
            e1.record(self.stream)
            (barrier or torch.cuda.synchronize)()
        return e0.elapsed_time(e1), clk

    def roofline(self, peaks, ms_kernel, ms_direct, clk):
        w = self.w
        fl = algorithmic_flops(w, self.iters, iterative_only=True)
        tf = fl / (ms_kernel * 1e-3) / 1e12
        traffic, src = NCU_TRAFFIC.get(int(w.name[3]), (None, None)) if w.name in [c.name for c in inputs.CONFIGS.values()] else (None, None)
        c = clk.summary()
        return {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": tf / peaks["bf16_tflops"], "traffic": traffic, "traffic_source": src,
                "kernel": f"iterative-rows forward kernel (forward_tc_kernel<{w.d}>)", "ms_per_launch": ms_kernel,
                "algorithmic_flops_per_launch": fl, "algorithmic_bytes_per_launch": int(self.set_bytes),
                "peak_source": f"{peaks['source']} burst bf16 (MEASURED_PEAKS.json)",
                "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": tf / 2250.0,
                "direct_rows_ms_per_launch": ms_direct, "sm_mhz": c["sm_mhz"],
                "ms_x_mhz": ms_kernel * c["sm_mhz"] if c["sm_mhz"] else None}

    def preconditioned(self, peaks, steps, warmup):
        """The same step with cg_precondition = 1 (inverse key covariance per block of 128 keys as CG preconditioner,
        built by a pre-pass inside the timed call): fewer iterations, so fewer algorithmic flops and less time."""
        w, L, torch = self.w, self.L, self.torch
        self.precondition = 1
        iters = torch.zeros((w.B, w.H, w.n), dtype=torch.int32, device="cuda")
        L.lla_forward_ex(*self.sets[0], self.outs[0], w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, causal=1, iters=iters,
                         workspace=self.ws, workspace_bytes=self.ws_bytes, stream=self.sp, cg_precondition=1)
        torch.cuda.synchronize()
        it = iters.cpu().numpy()
        ms, clk = self.timed(steps, warmup)
        self.precondition = 0
        ms /= steps
        fl = algorithmic_flops(w, it)
        cg = it[it >= 0]
        c = clk.summary()
        return {"ms_per_step": ms, "tokens_per_s": w.B * w.n / (ms * 1e-3), "cg_mean_iters": float(cg.mean()) if cg.size else 0.0,
                "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_bf16_peak_whole_step": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                "sm_mhz": c["sm_mhz"], "note": "optional mode (lla_forward_params.cg_precondition = 1); pre-pass kernels "
                "inside the timed step; flops count the iterations executed, which this mode roughly halves"}, clk

    def solver(self):
        L = self.L
        cg = self.iters[self.iters >= 0]
        return {"cg_tol": 1e-4, "cg_max_iters": 64, "cg_mean_iters": float(cg.mean()) if cg.size else 0.0,
                "cg_max_iters_seen": int(cg.max()) if cg.size else 0,
                "rows_at_iter_cap": int(self.status[L.STATUS_ROWS_AT_CAP]),
                "direct_rows_per_head": int((self.iters.reshape(-1, self.w.n)[0] < 0).sum())}


def measure_leg(L, torch, peaks, w, local, steps, warmup):
    """A prefill workload as a sub-object: whole step, dominant kernel alone, direct rows alone."""
    p = Prefill(L, torch, w, local)
    p.probe()
    ms_all, clk_all = p.timed(steps, warmup)
    ms_k, clk_k = p.timed(steps, 3, L.LLA_PHASE_ITERATIVE)
    ms_d, _ = p.timed(steps, 3, L.LLA_PHASE_DIRECT)
    ms_step = ms_all / steps
    c = clk_all.summary()
    pre, clk_p = p.preconditioned(peaks, max(10, steps // 2), 3)
    leg = {"config": workload_config(w), "steps": steps, "ms_per_step": ms_step, "preconditioned": pre,
           "tokens_per_s": w.B * w.n / (ms_step * 1e-3),
           "tflops": algorithmic_flops(w, p.iters) / (ms_step * 1e-3) / 1e12,
           "frac_of_bf16_peak_whole_step": algorithmic_flops(w, p.iters) / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
           "sm_mhz": c["sm_mhz"], "ms_x_mhz": ms_step * c["sm_mhz"] if c["sm_mhz"] else None,
           "roofline": p.roofline(peaks, ms_k / steps, ms_d / steps, clk_k), "solver": p.solver()}
    return leg, p, [clk_all, clk_k, clk_p]


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2510_01450_b200 as L

    world = env_int("WORLD_SIZE", 1)
    rank = env_int("RANK", 0)
    local = env_int("LOCAL_RANK", 0)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    peaks = load_peaks()
    base = inputs.CONFIGS[args.workload]
    w = base.shrink(seed=base.seed + 1000 * rank)
    if args.heads > 0:
        w = w.shrink(H=args.heads, name=f"{base.name}_H{args.heads}")
    samplers = []

    # ---- headline: device-resident throughput of the whole forward step ----
    head = Prefill(L, torch, w, local)
    head.probe()
    ms_total, clk = head.timed(args.steps, args.warmup, barrier=barrier)
    ms_total = max_over_ranks(ms_total)
    samplers.append(clk)
    c_head = clk.summary()
    # ---- dominant kernel alone (iterative rows) and the direct rows alone, per-launch average ----
    ms_kernel, clk_k = head.timed(args.steps, 3, L.LLA_PHASE_ITERATIVE)
    ms_direct, _ = head.timed(args.steps, 3, L.LLA_PHASE_DIRECT)
    samplers.append(clk_k)
    ms_kernel /= args.steps
    ms_direct /= args.steps

    pre_leg, clk_p = head.preconditioned(peaks, max(5, args.steps // 2), 3)
    samplers.append(clk_p)

    # ---- end to end through the host-buffer entry point (pinned memory) ----
    hq, hk, hv = head.host_bf16
    pq, pk, pv = (t.pin_memory() for t in (hq, hk, hv))
    pout = torch.empty((w.B, w.H, w.n, w.dv), dtype=torch.bfloat16).pin_memory()

    def e2e_step():
        L.lla_forward_host(pq, pk, pv, pout, w.B, w.H, w.n, w.d, w.dv, L.LLA_BF16, L.LLA_BF16, w.scale,
                           w.lam, 1, head.sp)

    for _ in range(3):
        e2e_step()
    e2e_steps = max(5, args.steps // 4)
    barrier()
    with ClockSampler(local) as clk_e:
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_s = max_over_ranks(time.perf_counter() - t0)
    samplers.append(clk_e)
    barrier()
    del pq, pk, pv

    # ---- the other prefill workloads, decode and backward: rank 0 only ----
    legs, decode, backward, parity = {}, None, None, {}
    leg_objs = {}
    if rank == 0 and not args.no_legs:
        for c in LEGS:
            if c == args.workload:
                continue
            wl = inputs.CONFIGS[c]
            est_ms = {2: 0.4, 3: 1.6}.get(c, 5.0)
            leg_steps = int(max(20, min(400, 300.0 / est_ms)))      # about 0.3 s per timed region
            leg, obj, cl = measure_leg(L, torch, peaks, wl, local, leg_steps, max(3, args.warmup))
            legs[f"prefill_cfg{c}"] = leg
            leg_objs[c] = obj
            samplers += cl
    if rank == 0 and not args.no_decode:
        decode, cl = bench_decode(L, torch, peaks, head.sp, head.stream, local)
        samplers.append(cl)
    backward3 = backward4 = None
    if rank == 0 and not args.no_backward:
        bw_obj = leg_objs.get(2) or Prefill(L, torch, inputs.CONFIGS[2], local)
        backward, cl = bench_backward(L, torch, peaks, bw_obj, local)
        samplers.append(cl)
        if 3 in leg_objs:      # the n = 4096 workload as well, where the pair kernels dominate the pass
            backward3, cl = bench_backward(L, torch, peaks, leg_objs[3], local, steps=10, nsets=2)
            samplers.append(cl)
        if head.w.name.startswith(inputs.CONFIGS[HEADLINE].name):      # and the headline workload (d = 128; also with --heads)
            backward4, cl = bench_backward(L, torch, peaks, head, local, steps=4, warmup=3, nsets=2)
            samplers.append(cl)

    tokens_step = w.B * w.n
    ms_step = ms_total / args.steps
    value = world * tokens_step / (ms_step * 1e-3)
    flops_step = algorithmic_flops(w, head.iters)
    roof = head.roofline(peaks, ms_kernel, ms_direct, clk_k)
    h2d = int(sum(t.numel() * 2 for t in (hq, hk, hv)))
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in/out, f32 accumulate", "data": "synthetic",
        "config": workload_config(w), "solver": head.solver(),
        "tflops": flops_step / (ms_step * 1e-3) / 1e12,
        "frac_of_bf16_peak_whole_step": flops_step / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "sm_mhz": c_head["sm_mhz"], "ms_x_mhz": ms_step * c_head["sm_mhz"] if c_head["sm_mhz"] else None,
        "roofline": roof, "preconditioned": pre_leg,
        "e2e": {"value": world * tokens_step * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": int(pout.numel() * 2), "steps": e2e_steps,
                "ms_per_step": 1e3 * e2e_s / e2e_steps,
                "note": "lla_forward_host on pinned buffers; the host link carries "
                        f"{(h2d + pout.numel() * 2) / 1e6:.0f} MB per step"},
        # per step: the fp16 copy of k, the iterative-rows kernel, the direct-rows kernel
        "gpu_launches": 3 * args.steps,
    }
    line.update(legs)
    if decode is not None:
        line["decode"] = decode
    if backward is not None:
        line["backward"] = backward
    if backward3 is not None:
        line["backward_cfg3"] = backward3
    if backward4 is not None:
        line["backward_cfg4"] = backward4
    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"], parity[f"cfg{args.workload}"] = cpu_baseline(head, 15.0)
            for c, obj in leg_objs.items():
                _, parity[f"cfg{c}"] = cpu_baseline(obj, 4.0)
            line["parity"] = parity
        line["clocks"] = merge_clocks(samplers)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def bench_decode(L, torch, peaks, sp, stream, local, steps=30, warmup=5):
    wd = inputs.CONFIGS[5]
    gen = torch.Generator(device="cuda").manual_seed(wd.seed)
    inv = 1.0 / np.sqrt(wd.d)
    kc = (torch.randn((wd.B, wd.H, wd.n, wd.d), generator=gen, device="cuda", dtype=torch.float32) * inv).to(torch.bfloat16)
    vc = torch.randn((wd.B, wd.H, wd.n, wd.dv), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    q = (torch.randn((wd.B, wd.H, wd.d), generator=gen, device="cuda", dtype=torch.float32) * inv).to(torch.bfloat16)
    lens_np = np.random.default_rng(wd.seed).integers(wd.len_min, wd.len_max + 1, size=wd.B).astype(np.int32)
    lens = torch.from_numpy(lens_np).cuda()
    out = torch.empty((wd.B, wd.H, wd.dv), dtype=torch.bfloat16, device="cuda")
    for _ in range(warmup):
        L.lla_decode(q, kc, vc, lens, out, wd.B, wd.H, wd.n, wd.d, wd.dv, wd.scale, wd.lam, sp)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clk:
        e0.record(stream)
        for _ in range(steps):
            L.lla_decode(q, kc, vc, lens, out, wd.B, wd.H, wd.n, wd.d, wd.dv, wd.scale, wd.lam, sp)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    live_bytes = float(lens_np.astype(np.int64).sum()) * wd.H * (wd.d + wd.dv) * 2
    gbs = live_bytes / (ms * 1e-3) / 1e9
    c = clk.summary()
    del kc, vc
    return {"workload": wd.name, "us_per_step": ms * 1e3, "us_per_token": ms * 1e3 / wd.B, "steps": steps,
            "sm_mhz": c["sm_mhz"], "ms_x_mhz": ms * c["sm_mhz"] if c["sm_mhz"] else None,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": NCU_DECODE_TRAFFIC[0],
                         "traffic_source": NCU_DECODE_TRAFFIC[1], "algorithmic_bytes": live_bytes,
                         "frac_of_nominal_8TBs": gbs / 8000.0,
                         "peak_source": f"{peaks['source']} copy bandwidth (MEASURED_PEAKS.json)"},
            "l2": "live cache bytes (1.2 GB) exceed L2 (126 MB)"}, clk


def bench_backward(L, torch, peaks, pre, local, steps=20, warmup=3, nsets=4):
    """Backward pass (gradients with respect to q, k, v) on the prefill workload of `pre`: the forward
    runs once per input set outside the timed region to save rho, stats and the fp32 output; the timed steps
    are lla_backward_ex alone, rotating over nsets sets of inputs and saved tensors (together larger than L2)."""
    w, sp, stream = pre.w, pre.sp, pre.stream
    shape = (w.B, w.H, w.n, w.d)
    g = torch.from_numpy(inputs.make_upstream_grad(w)).cuda()
    saved = []
    for r in range(nsets):
        q, k, v = pre.sets[r]
        out = torch.empty(shape, dtype=torch.float32, device="cuda")
        rho = torch.empty(shape, dtype=torch.float32, device="cuda")
        stats = torch.empty((w.B, w.H, w.n, 3), dtype=torch.float32, device="cuda")
        L.lla_forward_ex(q, k, v, out, w.B, w.H, w.n, w.d, w.dv, w.scale, w.lam, causal=1, out_dtype=L.LLA_F32,
                         rho=rho, stats=stats, stream=sp)
        saved.append((q, k, v, out, torch.roll(g, r, 1).contiguous(), rho, stats))
    grads = [torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(3)]
    nbytes = L.lla_backward_workspace_bytes(w.B, w.H, w.n, w.d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    iters = torch.full((w.B, w.H, w.n), -1, dtype=torch.int32, device="cuda")

    def step(i, **kw):
        L.lla_backward_ex(*saved[i % nsets], *grads, w.B, w.H, w.n, w.d, w.scale, w.lam, workspace=ws,
                          workspace_bytes=nbytes, stream=sp, **kw)

    step(0, iters=iters)
    torch.cuda.synchronize()
    it = iters.cpu().numpy().reshape(-1, w.n).astype(np.float64)
    pairs = np.arange(1, w.n + 1, dtype=np.float64)
    # per (query, key) pair: four score-like products and five output products (18 d) in the pair kernel, four
    # products (8 d) in the moments kernel, 6 d per executed CG iteration of the extra solve
    flops = float((26.0 * w.d * pairs[None, :] + 6.0 * w.d * pairs[None, :] * np.maximum(it, 0.0)).sum())
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clk:
        e0.record(stream)
        for i in range(steps):
            step(warmup + i)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    # the same steps with the extra solve preconditioned (optional mode, as in the forward)
    step(0, iters=iters, cg_precondition=1)
    torch.cuda.synchronize()
    it_pc = iters.cpu().numpy().reshape(-1, w.n).astype(np.float64)
    e0.record(stream)
    for i in range(steps):
        step(warmup + i, cg_precondition=1)
    e1.record(stream)
    torch.cuda.synchronize()
    ms_pc = e0.elapsed_time(e1) / steps
    set_bytes = sum(t.numel() * t.element_size() for t in saved[0])
    c = clk.summary()
    return {"workload": w.name, "ms_per_step": ms, "tokens_per_s": w.B * w.n / (ms * 1e-3),
            "tflops": flops / (ms * 1e-3) / 1e12,
            "frac_of_bf16_peak": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "roofline": {"bound": "tensor", "achieved": flops / (ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"], "traffic": None,
                         "kernel": "the whole pass (eight launches: solve, dK/dV, dQ, moments, direct rows, ...; profiles/backward_cfg3.md)",
                         "peak_source": f"{peaks['source']} burst bf16 (MEASURED_PEAKS.json)"},
            "cg_mean_iters": float(it[it >= 0].mean()) if (it >= 0).any() else 0.0,
            "preconditioned": {"ms_per_step": ms_pc, "cg_mean_iters": float(it_pc[it_pc >= 0].mean()) if (it_pc >= 0).any() else 0.0,
                               "note": "optional mode (lla_backward_params.cg_precondition = 1)"},
            "algorithmic_flops_per_step": flops, "gpu_launches_per_step": 8,
            "sm_mhz": c["sm_mhz"], "ms_x_mhz": ms * c["sm_mhz"] if c["sm_mhz"] else None,
            "l2": f"inputs and saved tensors rotate over {nsets} sets ({nsets * set_bytes / 1e6:.0f} MB > 126 MB L2)",
            "inputs": "bf16 q, k, v; fp32 upstream gradient, forward output, rho, stats; fp32 gradients"}, clk


def cpu_baseline(pre, budget_s):
    """The oracle, untuned, on this machine's host cores, on a bounded uniform row sample of the workload, and
    the parity figures of the device output (fp32 buffer) on those same rows."""
    from oracle import lla_oracle
    w = pre.w
    q, k, v = pre.host
    probe = oracle_sample_rows(w, 64, 7)
    t0 = time.perf_counter()
    lla_oracle.forward_rows(q, k, v, w.scale, w.lam, rows=probe)
    per_row = (time.perf_counter() - t0) / probe.size
    total = w.B * w.H * w.n
    n_rows = int(max(64, min(total, budget_s / max(per_row, 1e-9))))
    rows = oracle_sample_rows(w, n_rows, 8)
    t0 = time.perf_counter()
    ref = lla_oracle.forward_rows(q, k, v, w.scale, w.lam, rows=rows)
    dt = time.perf_counter() - t0
    got = pre.out32[rows].astype(np.float64)
    diff = got - ref
    e_row = np.linalg.norm(diff, axis=1) / np.linalg.norm(ref, axis=1)
    e_elem = np.abs(diff).max(axis=1) / np.abs(ref).max(axis=1)
    parity = {"rows": int(rows.size), "output": "fp32 buffer, bf16 inputs",
              "E_row_max": float(e_row.max()), "E_row_median": float(np.median(e_row)),
              "E_elem_max": float(e_elem.max()), "E_glob": float(np.abs(diff).max() / np.abs(ref).max()),
              "metrics": "E_row = |o_i - ref_i|_2 / |ref_i|_2; E_elem = |o_i - ref_i|_inf / |ref_i|_inf; "
                         "E_glob = max|o - ref| / max|ref|; gate 2e-3 on E_row"}
    base = {"value": rows.size / w.H / dt, "unit": UNIT, "cores": lla_oracle.threads(), "kind": "oracle",
            "sample": f"{rows.size} of {total} rows of {w.name}, drawn uniformly over (batch, head, position); "
                      f"{dt:.1f} s; tokens = rows / H"}
    return base, parity


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, choices=[2, 3, 4], default=HEADLINE,
                    help="prefill workload of the headline (default: the largest, n=16384, d=128)")
    ap.add_argument("--heads", type=int, default=0,
                    help="profiling aid: run the headline workload with this many heads (a small case of the same "
                         "kernel for an ncu capture; the line's config shows it)")
    ap.add_argument("--no-legs", action="store_true", help="skip the other prefill workloads")
    ap.add_argument("--no-decode", action="store_true", help="skip the decode measurement")
    ap.add_argument("--no-backward", action="store_true", help="skip the backward-pass measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing and parity figures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
