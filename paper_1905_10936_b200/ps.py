"""The paper's own setting on top of the C ABI: one worker per process/GPU and the server
sharded by block range over the same processes (Algorithm 2 / Algorithm 4 push and pull;
Section 4.2: more parameter servers relieve the server, and a block's signs and scale should
travel in one message).

Rank r of G is worker r (M = G) and the server of the block range `plan[r]`.  One iteration:

    engine.worker_step(0, grad)                       worker lines of Algorithm 4 (local)
    engine.pack_message(0, 0, B, send)                all blocks, fused [scale | words] per block
    all-to-all                                        rank q receives every worker's slice for plan[q]
    engine.server_step_range(b0, b1, recv)            server lines on the own block range
    engine.pack_message(-1, b0, b1, update_slice)
    all-gather                                        concatenated slices = the whole update
    engine.apply_update(0, B, update)                 x <- x - eta * update on every rank

This module only moves 32-bit buffers between ranks (torch.distributed collectives on tensors
that live in the receiving rank's own memory) and calls the engine; every arithmetic step runs
inside the engine.  The same orchestration runs (a) over a real process group (NCCL on GPUs,
gloo on CPU with a stand-in engine in the tests) and (b) with all ranks emulated one after the
other in a single process, where the "collectives" are slice copies between the ranks' buffers.

Push variant (no pack kernel, no collective on the data path): the kernels store the messages
where their readers are.  Every rank's receive and update buffers are mapped into its peers
(symmetric memory); the worker kernel writes block b's [scale | words] straight into the
receive buffer of the rank that serves b, and each server writes its update slice into every
rank's update buffer:

    engine.worker_step_push(0, grad, block_dst)       block_dst[b] = address inside server(b)'s recv
    barrier                                           all messages have landed
    engine.server_step_range(b0, b1, recv)
    engine.push_message(-1, b0, b1, update_dst)       the slice, stored into every rank's update
    barrier
    engine.apply_update(0, B, update)

Only plain stores cross the links; the barrier is a one-element all-reduce on the same stream
(no kernel of this package ever waits for another device).  Two barriers per iteration also
order the buffers' reuse: a rank starts its next worker step only after the second barrier,
i.e. after every server has finished reading the receive buffers of this iteration.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np
import torch

from .workloads import shard_blocks


@dataclass
class RangePlan:
    b0: int
    b1: int
    unit0: int      # where the range's slice starts in a message that covers all blocks
    units: int      # length of the slice in 32-bit units


def message_unit_offsets(sizes: Sequence[int]) -> np.ndarray:
    """unit[b] = start of block b in the fused message of all blocks (B+1 entries): each block
    takes one unit for its scale and ceil(d_b/32) units for its packed signs."""
    sizes = np.asarray(sizes, dtype=np.int64)
    return np.concatenate([[0], np.cumsum(1 + (sizes + 31) // 32)]).astype(np.int64)


def make_plan(sizes: Sequence[int], world: int) -> List[RangePlan]:
    """Block range served by each rank (whole blocks, balanced by element count) and where its
    slice sits in a whole-layout message."""
    unit = message_unit_offsets(sizes)
    plan = []
    for r in range(world):
        b0, b1 = shard_blocks(sizes, world, r)
        plan.append(RangePlan(b0, b1, int(unit[b0]), int(unit[b1] - unit[b0])))
    return plan


class Rank:
    """One worker + one server shard.  `engine` is an EFEngine created with
    one_local_worker=True and M = world (or any object with the same methods)."""

    def __init__(self, engine, sizes: Sequence[int], rank: int, world: int, device=None,
                 recv: Optional[torch.Tensor] = None, update: Optional[torch.Tensor] = None):
        """recv / update: buffers to use instead of fresh ones (e.g. symmetric memory), of
        recv_units(plan, rank) resp. total units int32 elements."""
        self.engine, self.rank, self.world = engine, rank, world
        self.sizes = [int(v) for v in sizes]
        self.B = len(sizes)
        self.plan = make_plan(sizes, world)
        self.mine = self.plan[rank]
        self.total_units = int(message_unit_offsets(sizes)[-1])
        dev = device if device is not None else getattr(engine, "device", "cpu")
        i32 = dict(dtype=torch.int32, device=dev)
        self.send = torch.zeros(self.total_units, **i32)                   # my message, all blocks
        width = recv_stride(self.plan, rank)
        if recv is None:
            recv = torch.zeros(world * width, **i32)
        if update is None:
            update = torch.zeros(self.total_units, **i32)
        assert recv.numel() >= world * width and update.numel() >= self.total_units
        self.recv = recv[:world * width].view(world, width)                # every worker's slice for my range
        self.update = update[:self.total_units]                            # the whole update
        self.block_dst = None      # push variant: device table of B addresses (connect_*)
        self.update_dst = None     # ... and where my update slice goes on every rank
        if engine is not None and self.mine.units > 0:
            assert engine.message_units(self.mine.b0, self.mine.b1) == self.mine.units
            assert engine.message_units(0, self.B) == self.total_units

    # ---- the compute calls, in protocol order ------------------------------------------------
    def work(self, grad) -> None:
        self.engine.worker_step(0, grad)
        self.engine.pack_message(0, 0, self.B, self.send)

    def serve(self) -> None:
        m = self.mine
        if m.b1 > m.b0:
            self.engine.server_step_range(m.b0, m.b1, self.recv)
            self.engine.pack_message(-1, m.b0, m.b1, self.update[m.unit0:m.unit0 + m.units])

    def apply(self) -> None:
        self.engine.apply_update(0, self.B, self.update)

    # ---- push variant ------------------------------------------------------------------------
    def connect(self, recv_ptrs: Sequence[int], update_ptrs: Sequence[int]) -> None:
        """recv_ptrs[q] / update_ptrs[q]: address, valid on THIS device, of rank q's receive /
        update buffer (its own memory for q == rank, a peer mapping otherwise)."""
        table = push_table(self.sizes, self.plan, self.rank, recv_ptrs)
        self.block_dst = torch.from_numpy(table).to(self.update.device)
        self.update_dst = [int(p) + 4 * self.mine.unit0 for p in update_ptrs]

    def work_push(self, grad) -> None:
        self.engine.worker_step_push(0, grad, self.block_dst)

    def serve_push(self) -> None:
        m = self.mine
        if m.b1 > m.b0:
            self.engine.server_step_range(m.b0, m.b1, self.recv)
            self.engine.push_message(-1, m.b0, m.b1, self.update_dst)


def recv_stride(plan: List[RangePlan], q: int) -> int:
    """Row length (32-bit units) of rank q's receive buffer: row i holds worker i's slice."""
    return max(plan[q].units, 1)


def push_table(sizes: Sequence[int], plan: List[RangePlan], rank: int,
               recv_ptrs: Sequence[int]) -> np.ndarray:
    """dst[b] = where worker `rank` stores block b's fused message: row `rank` of the receive
    buffer of the rank that serves b, at the block's place in that rank's range (bytes)."""
    unit = message_unit_offsets(sizes)
    dst = np.zeros(len(sizes), dtype=np.int64)
    for q, p in enumerate(plan):
        row = int(recv_ptrs[q]) + 4 * rank * recv_stride(plan, q)
        for b in range(p.b0, p.b1):
            dst[b] = row + 4 * int(unit[b] - unit[p.b0])
    return dst


# ---------------------------------------------------------------------------- real process group
def exchange_messages(rk: Rank, group=None) -> None:
    """All-to-all: my slice for plan[q] goes to rank q; I receive every worker's slice for my range."""
    import torch.distributed as dist
    u = rk.mine.units
    out = rk.recv.view(-1)[:rk.world * u]               # row i of recv = worker i's slice
    dist.all_to_all_single(out, rk.send, output_split_sizes=[u] * rk.world,
                           input_split_sizes=[p.units for p in rk.plan], group=group)


def gather_update(rk: Rank, group=None) -> None:
    """All-gather of the servers' update slices (padded to equal length for the collective,
    then laid end to end in block order)."""
    import torch.distributed as dist
    width = max(max(p.units for p in rk.plan), 1)
    mine = torch.zeros(width, dtype=torch.int32, device=rk.update.device)
    m = rk.mine
    mine[:m.units].copy_(rk.update[m.unit0:m.unit0 + m.units])
    everyone = torch.empty(rk.world * width, dtype=torch.int32, device=rk.update.device)
    dist.all_gather_into_tensor(everyone, mine, group=group)
    for q, p in enumerate(rk.plan):
        if q != rk.rank and p.units:
            rk.update[p.unit0:p.unit0 + p.units].copy_(everyone[q * width:q * width + p.units])


def step(rk: Rank, grad, group=None) -> None:
    """One iteration of rank `rk.rank` inside a process group."""
    rk.work(grad)
    exchange_messages(rk, group)
    rk.serve()
    gather_update(rk, group)
    rk.apply()


def symmetric_buffers(sizes: Sequence[int], rank: int, world: int, device, group=None):
    """Receive and update buffers of one rank in symmetric memory (every rank allocates the same
    size and maps its peers' copies).  Returns (recv, update, recv_ptrs, update_ptrs) for
    Rank(..., recv=, update=) and Rank.connect.  Fails loudly where symmetric memory is not
    available; the collective variant (step) needs none."""
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm
    plan = make_plan(sizes, world)
    total = int(message_unit_offsets(sizes)[-1])
    n_recv = (world * max(recv_stride(plan, q) for q in range(world)) + 3) // 4 * 4
    buf = symm.empty(n_recv + total, dtype=torch.int32, device=device)
    handle = symm.rendezvous(buf, dist.group.WORLD if group is None else group)
    buf.zero_()
    base = [int(p) for p in handle.buffer_ptrs]
    assert len(base) == world and base[rank] == buf.data_ptr()
    return buf[:n_recv], buf[n_recv:], base, [p + 4 * n_recv for p in base]


def stream_barrier(flag: torch.Tensor, group=None) -> None:
    """Every rank's work enqueued so far has finished before anything enqueued after this call
    starts on any rank: a one-element all-reduce on the current stream."""
    import torch.distributed as dist
    dist.all_reduce(flag, group=group)


def step_push(rk: Rank, grad, flag: torch.Tensor, group=None) -> None:
    """One iteration of rank `rk.rank` inside a process group, push variant (rk.connect first)."""
    rk.work_push(grad)
    stream_barrier(flag, group)
    rk.serve_push()
    stream_barrier(flag, group)
    rk.apply()


# ---------------------------------------------------------------------------- one-process emulation
def connect_emulated(ranks: List[Rank]) -> None:
    """Push variant with all ranks on one device: the peers' buffers are ordinary local tensors."""
    recv_ptrs = [r.recv.data_ptr() for r in ranks]
    update_ptrs = [r.update.data_ptr() for r in ranks]
    for r in ranks:
        r.connect(recv_ptrs, update_ptrs)


def step_emulated_push(ranks: List[Rank], grads: Sequence) -> None:
    """One iteration of all ranks, push variant, one after the other on one stream (stream order
    stands in for the barriers)."""
    for rk, g in zip(ranks, grads):
        rk.work_push(g)
    for rk in ranks:
        rk.serve_push()
    for rk in ranks:
        rk.apply()


def step_emulated(ranks: List[Rank], grads: Sequence) -> None:
    """The same iteration with all ranks held by ONE process and run one after the other; the
    collectives become slice copies between the ranks' buffers (no rank ever waits for another,
    so this is safe on a single device)."""
    for rk, g in zip(ranks, grads):
        rk.work(g)
    for dst in ranks:                                  # all-to-all
        m = dst.mine
        for src in ranks:
            if m.units:
                dst.recv[src.rank, :m.units].copy_(src.send[m.unit0:m.unit0 + m.units])
    for rk in ranks:
        rk.serve()
    for dst in ranks:                                  # all-gather
        for src in ranks:
            p = src.mine
            if src is not dst and p.units:
                dst.update[p.unit0:p.unit0 + p.units].copy_(src.update[p.unit0:p.unit0 + p.units])
    for rk in ranks:
        rk.apply()


# ---------------------------------------------------------------------------- host-side decoding
def unpack_message(msg: np.ndarray, sizes: Sequence[int], b0: int, b1: int):
    """(scales[b1-b0] float32, words uint32 of the range in the plain layout) from a fused message."""
    msg = np.ascontiguousarray(msg).view(np.uint32)
    unit = message_unit_offsets(sizes)
    scales, words = [], []
    for b in range(b0, b1):
        u = int(unit[b] - unit[b0])
        nw = (int(sizes[b]) + 31) // 32
        scales.append(msg[u:u + 1].view(np.float32)[0])
        words.append(msg[u + 1:u + 1 + nw])
    return np.array(scales, dtype=np.float32), (np.concatenate(words) if words else np.zeros(0, np.uint32))


def pack_message(scales: np.ndarray, words: np.ndarray, sizes: Sequence[int], b0: int, b1: int) -> np.ndarray:
    """Inverse of unpack_message (host side; the device side is ef_pack_message)."""
    out, w = [], 0
    for k, b in enumerate(range(b0, b1)):
        nw = (int(sizes[b]) + 31) // 32
        out.append(np.array([scales[k]], dtype=np.float32).view(np.uint32))
        out.append(np.asarray(words[w:w + nw], dtype=np.uint32))
        w += nw
    return np.concatenate(out) if out else np.zeros(0, np.uint32)
