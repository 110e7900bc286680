"""The cut-block exchange of paper_1905_10936_b200/sharded.py over a real process group (gloo,
CPU, world 2 and 3): the product's element sharding (workloads.shard_elements), its mapping of
local pieces to blocks and its all-reduce of per-block fp64 sums, with the oracle supplying the
numbers behind the engine interface.  After the first worker step every rank's completed scale
of every block must be the scale the unsharded oracle computes for the whole block."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.sharded import DistributedShard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class OraclePieces:
    """Engine stand-in on the host: the oracle's worker lines on this rank's local layout.  For a
    piece of a cut block the oracle's own scale is that of the piece alone, so the stand-in
    exposes what the library exposes: the piece's fp64 sum of |p| and a completed scale."""

    device = "cpu"

    def __init__(self, shard, M, mu, eta):
        from oracle import Oracle
        self.off = np.concatenate([[0], np.cumsum(shard.local_sizes)]).astype(np.int64)
        self.B, self.M = len(shard.local_sizes), M
        self.full = np.asarray(shard.full_sizes, dtype=np.int64)
        self.partial = self.full != np.diff(self.off)
        self.orc = Oracle(self.off, M, mu, eta) if self.B else None
        self.sums = np.zeros((M, self.B))
        self.scales = np.zeros((M, self.B), dtype=np.float32)
        self.ctx = True

    def worker_step_all(self, grads):
        for i in range(self.M):
            self.orc.worker_step(i, grads[i].numpy())
            p = np.abs(self.orc.last_p.astype(np.float64))
            self.sums[i] = np.add.reduceat(p, self.off[:-1])
            self.scales[i] = self.orc.scales(i)               # right for blocks held whole

    def block_sums(self, who, dst):
        dst[:self.B] = torch.from_numpy(np.where(self.partial, self.sums[who], 0.0))

    def complete_scales(self, who, totals):
        t = totals[:self.B].numpy()
        self.scales[who] = np.where(self.partial, (t / self.full).astype(np.float32), self.scales[who])


def _rank_main(rank, world, port, sizes, M, out):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.custom_workload("cut-gloo", sizes, M, scale_range=(1e-2, 1.0), config_id=79)
        ds = DistributedShard(w.sizes, M, w.mu, w.eta, rank, world,
                              make_engine=lambda sh, M, mu, eta: OraclePieces(sh, M, mu, eta))
        es = w.element_scales("cpu")
        lo, hi = ds.shard.elem_lo, ds.shard.elem_hi
        grads = torch.stack([w.draw_grad(0, i, "cpu", es)[lo:hi] for i in range(M)])
        ds.worker_step_all(grads)
        out[rank] = (ds.shard.global_block, ds.eng.scales.copy(), ds.any_cut, (lo, hi))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,sizes", [(2, [40960 + 64, 700, 8192]), (3, [40960 + 64, 700, 8192]),
                                         (3, [500, 600, 700])])      # blocks below the granule: never cut
def test_completed_scales_equal_the_whole_block_scales(world, sizes):
    from oracle import Oracle
    M = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), sizes, M, out), nprocs=world, join=True)
    w = wl.custom_workload("cut-gloo", sizes, M, scale_range=(1e-2, 1.0), config_id=79)
    es = w.element_scales("cpu")
    ref = Oracle(w.offsets, M, w.mu, w.eta)
    for i in range(M):
        ref.worker_step(i, w.draw_grad(0, i, "cpu", es).numpy())
    covered = 0
    for r in range(world):
        blocks, scales, any_cut, (lo, hi) = out[r]
        covered += hi - lo
        assert any_cut == any(l != f for q in range(world)
                              for l, f in zip(*(lambda s: (s.local_sizes, s.full_sizes))(
                                  wl.shard_elements(sizes, world, q))))
        for i in range(M):
            want = ref.scales(i)[blocks]
            assert np.all(np.abs(scales[i] - want) <= 1.2e-7 * want), (r, i, scales[i], want)
    assert covered == sum(sizes)


def test_element_shards_tile_the_vector_and_cut_on_word_boundaries():
    for sizes in ([40960 + 64, 700, 8192], wl.gpt2_medium_sizes(), wl.resnet50_sizes(), [5], [4096] * 7):
        for world in (1, 2, 3, 8):
            prev = 0
            for r in range(world):
                sh = wl.shard_elements(sizes, world, r)
                assert sh.elem_lo == prev
                prev = sh.elem_hi
                assert sum(sh.local_sizes) == sh.elem_hi - sh.elem_lo
                for l, f, o in zip(sh.local_sizes, sh.full_sizes, sh.offset_in_block):
                    assert o % 32 == 0 and o + l <= f            # pieces start on word boundaries
            assert prev == sum(sizes)
    with pytest.raises(ValueError):
        wl.shard_elements([100], 2, 0, granule=48)
