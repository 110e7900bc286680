"""Block-range sharding over ranks (the N > 1 path): two gloo ranks on CPU.

Every operation of the method is per element or per block, so a rank that owns whole blocks
needs no exchange.  Each rank runs the oracle on its own block range; the gathered shards must
equal the unsharded run bit for bit.  No GPU is involved.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_10936_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, sizes, M, steps, out):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    from oracle import Oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.custom_workload("shard", sizes, M, steps=steps, scale_range=(1e-2, 1.0), config_id=77)
        b0, b1 = wl.shard_blocks(w.sizes, world, rank)
        lo, hi = int(w.offsets[b0]), int(w.offsets[b1])
        sub_off = w.offsets[b0:b1 + 1] - w.offsets[b0]
        es = w.element_scales("cpu")
        orc = Oracle(sub_off, M, w.mu, w.eta) if b1 > b0 else None
        for t in range(steps):
            for i in range(M):
                g = w.draw_grad(t, i, "cpu", es).numpy()      # same seeded gradient on every rank
                if orc is not None:
                    orc.worker_step(i, g[lo:hi])
            if orc is not None:
                orc.server_step()
        # gather the shards of x and of the server scales on every rank (variable sizes)
        x_local = torch.from_numpy(orc.x.copy()) if orc is not None else torch.empty(0)
        s_local = torch.from_numpy(orc.scales(-1).copy()) if orc is not None else torch.empty(0)
        xs, ss = [None] * world, [None] * world
        dist.all_gather_object(xs, x_local)
        dist.all_gather_object(ss, s_local)
        tmax = torch.tensor([float(rank)])
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)               # the bench's max-over-ranks step
        if rank == 0:
            out["x"] = torch.cat(xs).numpy()
            out["scales"] = torch.cat(ss).numpy()
            out["tmax"] = float(tmax.item())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_block_range_shards_equal_the_unsharded_run(world):
    from oracle import Oracle
    sizes, M, steps = [700, 33, 4096, 10, 2500, 64, 1200], 3, 3
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), sizes, M, steps, out), nprocs=world, join=True)
    w = wl.custom_workload("shard", sizes, M, steps=steps, scale_range=(1e-2, 1.0), config_id=77)
    es = w.element_scales("cpu")
    ref = Oracle(w.offsets, M, w.mu, w.eta)
    for t in range(steps):
        for i in range(M):
            ref.worker_step(i, w.draw_grad(t, i, "cpu", es).numpy())
        ref.server_step()
    assert np.array_equal(out["x"], ref.x)
    assert np.array_equal(out["scales"], ref.scales(-1))
    assert out["tmax"] == world - 1


def test_shards_are_balanced_for_the_bench_layout():
    w = wl.make_workload(4)
    for world in (2, 4, 8):
        sizes = [sum(w.sizes[b0:b1]) for b0, b1 in
                 (wl.shard_blocks(w.sizes, world, r) for r in range(world))]
        assert sum(sizes) == w.d and max(sizes) == min(sizes)
