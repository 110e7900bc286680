"""The exchange logic of the sharded parameter server (paper_1905_10936_b200/ps.py) over a real
process group: gloo ranks on CPU, world 2 and 3.

The collectives, the slicing of the fused messages and the call sequence are the product's
(ps.step, ps.make_plan); the arithmetic behind the engine interface is supplied by the CPU
oracle (a worker oracle per rank, a server oracle per block range fed with the received
messages), so no GPU is involved.  Every rank must end with the parameters of one unsharded
oracle run, bit for bit."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_10936_b200 import ps
from paper_1905_10936_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class OracleRankEngine:
    """The engine interface ps.Rank needs, computed by the oracle on the host."""

    device = "cpu"

    def __init__(self, sizes, G, rank, mu, eta):
        from oracle import Oracle
        self.sizes = list(sizes)
        self.off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
        self.B, self.M, self.eta = len(sizes), G, np.float32(eta)
        self.worker = Oracle(self.off, 1, mu, eta)               # this rank's worker lines
        self.b0, self.b1 = wl.shard_blocks(sizes, G, rank)
        self.server = (Oracle(self.off[self.b0:self.b1 + 1] - self.off[self.b0], G, mu, eta)
                       if self.b1 > self.b0 else None)           # server lines on the own range
        self.x = np.zeros(int(self.off[-1]), dtype=np.float32)

    def message_units(self, b0, b1):
        u = ps.message_unit_offsets(self.sizes)
        return int(u[b1] - u[b0])

    def worker_step(self, i, grad):
        assert i == 0
        self.worker.worker_step(0, grad)
        self._msg = (self.worker.scales(0).copy(), self.worker.words(0).copy())
        self.worker.server_step()                                # only to reopen the oracle's iteration

    def pack_message(self, who, b0, b1, dst):
        woff = np.concatenate([[0], np.cumsum([(s + 31) // 32 for s in self.sizes])])
        if who == 0:
            sc, wd = self._msg[0][b0:b1], self._msg[1][woff[b0]:woff[b1]]
        else:
            assert (b0, b1) == (self.b0, self.b1)
            sc, wd = self.server.scales(-1), self.server.words(-1)
        out = ps.pack_message(sc, wd, self.sizes, b0, b1)
        dst.numpy().view(np.uint32)[:out.size] = out

    # push variant: `heap` is the address space all ranks share (a file every rank has mapped);
    # a destination address is a byte offset into it
    heap = None

    def _message(self, who, b0, b1):
        tmp = torch.zeros(self.message_units(b0, b1), dtype=torch.int32)
        self.pack_message(who, b0, b1, tmp)
        return tmp.numpy()

    def worker_step_push(self, i, grad, block_dst):
        self.worker_step(i, grad)
        for b, addr in enumerate(block_dst.tolist()):
            assert addr % 4 == 0
            msg = self._message(0, b, b + 1)
            self.heap[addr // 4:addr // 4 + msg.size] = msg

    def push_message(self, who, b0, b1, dst_ptrs):
        msg = self._message(who, b0, b1)
        for addr in dst_ptrs:
            self.heap[addr // 4:addr // 4 + msg.size] = msg

    def server_step_range(self, b0, b1, msgs):
        assert (b0, b1) == (self.b0, self.b1)
        zero = np.zeros(self.server.d, dtype=np.float32)
        for i in range(self.M):
            sc, wd = ps.unpack_message(msgs[i].numpy(), self.sizes, b0, b1)
            self.server.worker_step(i, zero)                     # opens slot i; its content is replaced
            self.server.scales(i)[:] = sc                        # by the message that arrived
            self.server.words(i)[:] = wd
        self.server.server_step()

    def apply_update(self, b0, b1, update):
        sc, wd = ps.unpack_message(update.numpy(), self.sizes, b0, b1)
        w = 0
        for k, b in enumerate(range(b0, b1)):
            n = self.sizes[b]
            bits = np.unpackbits(wd[w:w + (n + 31) // 32].view(np.uint8), bitorder="little")[:n].astype(bool)
            step = self.eta * sc[k]                               # binary32 product
            seg = self.x[self.off[b]:self.off[b + 1]]
            seg[:] = np.where(bits, seg + step, seg - step)
            w += (n + 31) // 32


def _rank_main(rank, world, port, sizes, steps, out):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.custom_workload("ps-gloo", sizes, world, steps=steps, scale_range=(1e-2, 1.0), config_id=78)
        eng = OracleRankEngine(w.sizes, world, rank, w.mu, w.eta)
        rk = ps.Rank(eng, w.sizes, rank, world, device="cpu")
        es = w.element_scales("cpu")
        for t in range(steps):
            ps.step(rk, w.draw_grad(t, rank, "cpu", es).numpy())
        out[rank] = (eng.x.copy(), (eng.b0, eng.b1),
                     eng.server.residual(-1).copy() if eng.server is not None else None)
    finally:
        dist.destroy_process_group()


def _heap_layout(sizes, world):
    """(units per rank, offset of the update buffer inside a rank's part): every rank's receive
    rows and update buffer, one rank after the other, in one shared file."""
    plan = ps.make_plan(sizes, world)
    n_recv = world * max(ps.recv_stride(plan, q) for q in range(world))
    return n_recv + int(ps.message_unit_offsets(sizes)[-1]), n_recv


def _rank_main_push(rank, world, port, sizes, steps, out, heap_path):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.custom_workload("ps-gloo", sizes, world, steps=steps, scale_range=(1e-2, 1.0), config_id=78)
        per_rank, n_recv = _heap_layout(w.sizes, world)
        heap = np.memmap(heap_path, dtype=np.int32, mode="r+", shape=(world * per_rank,))
        eng = OracleRankEngine(w.sizes, world, rank, w.mu, w.eta)
        eng.heap = heap
        mine = torch.from_numpy(heap[rank * per_rank:(rank + 1) * per_rank])
        rk = ps.Rank(eng, w.sizes, rank, world, device="cpu", recv=mine[:n_recv], update=mine[n_recv:])
        rk.connect([4 * q * per_rank for q in range(world)], [4 * (q * per_rank + n_recv) for q in range(world)])
        flag = torch.zeros(1)
        es = w.element_scales("cpu")
        for t in range(steps):
            ps.step_push(rk, w.draw_grad(t, rank, "cpu", es).numpy(), flag)
        out[rank] = (eng.x.copy(), (eng.b0, eng.b1),
                     eng.server.residual(-1).copy() if eng.server is not None else None)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("variant", ["collective", "push"])
@pytest.mark.parametrize("world,sizes", [(2, [700, 33, 4096, 10, 2500, 64, 1200]),
                                         (3, [700, 33, 4096, 10, 2500, 64, 1200]),
                                         (3, [100, 5000])])          # one rank serves no block
def test_sharded_server_over_gloo_equals_the_unsharded_oracle(world, sizes, variant, tmp_path):
    """collective: all-to-all and all-gather move the messages.  push: every rank stores its
    messages directly into the others' buffers (a file all ranks have mapped stands in for peer
    memory) and the only collectives are the two barriers per iteration."""
    from oracle import Oracle
    steps = 3
    mgr = mp.Manager()
    out = mgr.dict()
    if variant == "push":
        per_rank, _ = _heap_layout(sizes, world)
        heap_path = str(tmp_path / "heap.bin")
        np.zeros(world * per_rank, dtype=np.int32).tofile(heap_path)
        mp.spawn(_rank_main_push, args=(world, _free_port(), sizes, steps, out, heap_path), nprocs=world, join=True)
    else:
        mp.spawn(_rank_main, args=(world, _free_port(), sizes, steps, out), nprocs=world, join=True)
    w = wl.custom_workload("ps-gloo", sizes, world, steps=steps, scale_range=(1e-2, 1.0), config_id=78)
    es = w.element_scales("cpu")
    ref = Oracle(w.offsets, world, w.mu, w.eta)
    for t in range(steps):
        for i in range(world):
            ref.worker_step(i, w.draw_grad(t, i, "cpu", es).numpy())
        ref.server_step()
    for r in range(world):
        x, (b0, b1), resid = out[r]
        assert np.array_equal(x, ref.x), f"rank {r}: parameters differ from the unsharded run"
        if b1 > b0:
            lo, hi = int(w.offsets[b0]), int(w.offsets[b1])
            assert np.array_equal(resid, ref.residual(-1)[lo:hi])


def test_plan_slices_tile_the_whole_message():
    sizes = [700, 33, 4096, 10, 2500, 64, 1200]
    unit = ps.message_unit_offsets(sizes)
    assert unit[-1] == sum(1 + (s + 31) // 32 for s in sizes)
    for world in (1, 2, 3, 5, 9):
        plan = ps.make_plan(sizes, world)
        assert plan[0].b0 == 0 and plan[-1].b1 == len(sizes)
        assert all(a.b1 == b.b0 and a.unit0 + a.units == b.unit0 for a, b in zip(plan, plan[1:]))
        assert sum(p.units for p in plan) == unit[-1]
    sc = np.array([0.5, 2.0], dtype=np.float32)
    # blocks of 33 and 10 elements: 2 words and 1 word, each behind its block's scale
    msg = ps.pack_message(sc, np.arange(2 + 1, dtype=np.uint32), [33, 10], 0, 2)
    assert msg.size == 2 + 3 and msg[0] == np.float32(0.5).view(np.uint32) and msg[3] == np.float32(2.0).view(np.uint32)
    s2, w2 = ps.unpack_message(msg, [33, 10], 0, 2)
    assert np.array_equal(s2, sc) and np.array_equal(w2, np.arange(3, dtype=np.uint32))


def test_push_table_addresses():
    """Block b of worker r goes to row r of the receive buffer of the rank that serves b, at the
    block's place inside that rank's range."""
    sizes = [700, 33, 4096, 10, 2500, 64, 1200]
    unit = ps.message_unit_offsets(sizes)
    for world in (1, 2, 3, 9):
        plan = ps.make_plan(sizes, world)
        bases = [1 << 20 | (q << 32) for q in range(world)]          # distinct, 4-byte aligned
        seen = set()
        for r in range(world):
            table = ps.push_table(sizes, plan, r, bases)
            for q, p in enumerate(plan):
                for b in range(p.b0, p.b1):
                    rel = (int(table[b]) - bases[q]) // 4
                    row, col = divmod(rel, ps.recv_stride(plan, q))
                    assert row == r and col == unit[b] - unit[p.b0]
                    assert col + 1 + (sizes[b] + 31) // 32 <= ps.recv_stride(plan, q)   # stays inside its row
                    span = (int(table[b]), int(table[b]) + 4 * (1 + (sizes[b] + 31) // 32))
                    assert span not in seen
                    seen.add(span)
        # no two messages overlap
        spans = sorted(seen)
        assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:]))
