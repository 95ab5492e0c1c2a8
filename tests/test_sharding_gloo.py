"""The multi-GPU path shards independent (batch, head) units across ranks with no data-path
collective.  This CPU test runs that host logic with two gloo ranks: each rank takes its contiguous
share of the units, computes them (with the oracle standing in for the device), and the gathered
result must equal the unsharded one; the timing reduction (max over ranks) is exercised too."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_01450_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q, k, v, scale, lam, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import lla_oracle
    B, H, n, d = q.shape
    units = B * H
    lo, hi = inputs.shard_units(units, rank, world)
    qf, kf, vf = (x.reshape(1, units, n, -1) for x in (q, k, v))
    part = lla_oracle.forward(qf[:, lo:hi], kf[:, lo:hi], vf[:, lo:hi], scale, lam)[0]
    full = torch.zeros((units, n, v.shape[-1]), dtype=torch.float64)
    full[lo:hi] = torch.from_numpy(part)
    dist.all_reduce(full)                                  # test-side gather only; the product path has none
    t = torch.tensor([1.0 + rank], dtype=torch.float64)    # per-rank "elapsed"
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        ret["out"] = full.numpy()
        ret["tmax"] = float(t.item())
    dist.destroy_process_group()


def test_two_rank_sharding_matches_single_process(oracle):
    w = inputs.CONFIGS[2].shrink(B=1, H=3, n=48, d=16, dv=16, seed=21)   # 3 units over 2 ranks: uneven split
    q, k, v = inputs.make_prefill(w)
    want = oracle.forward(q, k, v, w.scale, w.lam).reshape(3, 48, 16)
    mgr = mp.Manager()
    ret = mgr.dict()
    port = _free_port()
    mp.spawn(_worker, args=(2, port, q, k, v, w.scale, w.lam, ret), nprocs=2, join=True)
    np.testing.assert_array_equal(ret["out"], want)
    assert ret["tmax"] == 2.0


def test_shard_units_partition():
    for units, world in ((32, 8), (7, 3), (2, 4), (1024, 6)):
        spans = [inputs.shard_units(units, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == units
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= 1
