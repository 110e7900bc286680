"""One layout cut by element count over several devices, blocks included (the simulated-workers
build's own way to scale: every rank holds ALL M workers' state for its element range).

Every operation of the method is per element except the block's L1 norm (Section 3.2), so the
only exchange is one fp64 number per cut block and call: each rank's partial sum of |p| over
its piece, added up over the ranks (an all-reduce of B doubles), after which every rank forms
the same scale.  A rank whose range holds only whole blocks exchanges zeros.

`ShardedEngine` drives R rank engines that all live in this process, one after the other (the
"all-reduce" is then a sum over the ranks' buffers): that is how the cut is tested on a single
GPU.  `DistributedShard` is the same iteration for one rank of a torch.distributed group.
Both only move B-double buffers and call the engine; all arithmetic runs in the library.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from .engine import EFEngine
from .workloads import ElementShard, shard_elements


def _make_rank_engine(shard: ElementShard, M: int, mu: float, eta: float, **kw) -> EFEngine:
    offsets = np.concatenate([[0], np.cumsum(shard.local_sizes)]).astype(np.int64)
    eng = EFEngine(offsets, M, mu, eta, **kw)
    if any(l != f for l, f in zip(shard.local_sizes, shard.full_sizes)):
        eng.set_block_divisors(shard.full_sizes)
    return eng


class _RankState:
    def __init__(self, shard: ElementShard, num_blocks: int, eng: EFEngine):
        self.shard, self.eng = shard, eng
        self.gidx = torch.tensor(shard.global_block, dtype=torch.int64, device=eng.device)
        self.local = torch.zeros(max(eng.B, 1), dtype=torch.float64, device=eng.device)     # per local block
        self.globl = torch.zeros(num_blocks, dtype=torch.float64, device=eng.device)        # per block of the whole layout

    def sums_to_global(self, who: int) -> torch.Tensor:
        """This rank's contribution to every block's L1 sum (zeros for blocks it holds whole)."""
        self.eng.block_sums(who, self.local)
        self.globl.zero_()
        self.globl.index_add_(0, self.gidx, self.local[:self.eng.B])
        return self.globl

    def complete(self, who: int, totals: torch.Tensor) -> None:
        self.local[:self.eng.B].copy_(totals[self.gidx])
        self.eng.complete_scales(who, self.local)


class ShardedEngine:
    """R element-range shards of one layout on one device, stepped one after the other; has
    the parts of EFEngine's interface the parity protocol uses (whole-vector views are gathered)."""

    def __init__(self, offsets, M: int, mu: float, eta: float, ranks: int = 2, granule: int = 4096,
                 scale_mode: str = "auto", weight_decay: bool = False, diagnostics: bool = False):
        assert not diagnostics, "per-block diagnostics are not defined for pieces of blocks"
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        self.sizes = np.diff(self.offsets).tolist()
        self.B, self.d, self.M = len(self.sizes), int(self.offsets[-1]), int(M)
        self.ranks: List[_RankState] = []
        for r in range(ranks):
            sh = shard_elements(self.sizes, ranks, r, granule)
            if sh.elem_hi > sh.elem_lo:
                eng = _make_rank_engine(sh, M, mu, eta, scale_mode=scale_mode, weight_decay=weight_decay)
                self.ranks.append(_RankState(sh, self.B, eng))
        self.device = self.ranks[0].eng.device
        self.cut = any(rk.eng.B and any(l != f for l, f in zip(rk.shard.local_sizes, rk.shard.full_sizes))
                       for rk in self.ranks)

    # ---- the exchange: a sum over the ranks' B-double buffers ---------------------------------
    def _reduce_and_complete(self, who: int) -> None:
        if not self.cut:
            return
        total = torch.zeros(self.B, dtype=torch.float64, device=self.device)
        for rk in self.ranks:
            total += rk.sums_to_global(who)
        for rk in self.ranks:
            if rk.eng.ctx and any(l != f for l, f in zip(rk.shard.local_sizes, rk.shard.full_sizes)):
                rk.complete(who, total)

    # ---- steps -----------------------------------------------------------------------------
    def worker_step(self, i: int, grad: torch.Tensor) -> None:
        for rk in self.ranks:
            g = grad[rk.shard.elem_lo:rk.shard.elem_hi]
            rk.eng.worker_step(i, g if g.data_ptr() % 16 == 0 else g.clone())
        self._reduce_and_complete(i)

    def worker_step_all(self, grads: torch.Tensor) -> None:
        for rk in self.ranks:
            n = rk.shard.elem_hi - rk.shard.elem_lo
            stride = (n + 3) // 4 * 4
            local = torch.zeros(self.M, stride, dtype=torch.float32, device=self.device)
            local[:, :n].copy_(grads[:, rk.shard.elem_lo:rk.shard.elem_hi])
            rk.eng.worker_step_all(local)
        for i in range(self.M):
            self._reduce_and_complete(i)

    def server_step(self) -> None:
        for rk in self.ranks:
            rk.eng.server_step_range(0, rk.eng.B)
        self._reduce_and_complete(-1)
        for rk in self.ranks:
            rk.eng.apply_update(0, rk.eng.B)

    def set_eta(self, eta: float) -> None:
        for rk in self.ranks:
            rk.eng.set_eta(eta)

    def set_weight_decay(self, lam: float) -> None:
        for rk in self.ranks:
            rk.eng.set_weight_decay(lam)

    # ---- whole-vector views (gathered copies) --------------------------------------------------
    def _cat(self, fn) -> torch.Tensor:
        return torch.cat([fn(rk.eng) for rk in self.ranks])

    def params(self) -> torch.Tensor:
        return _Gathered(self, lambda e: e.params())

    def decay_momentum(self) -> torch.Tensor:
        return self._cat(lambda e: e.decay_momentum())

    def momentum(self, i: int) -> torch.Tensor:
        return self._cat(lambda e: e.momentum(i))

    def residual(self, i: int = -1) -> torch.Tensor:
        return self._cat(lambda e: e.residual(i))

    def worker_words(self, i: int) -> torch.Tensor:
        return self._cat(lambda e: e.worker_words(i))      # pieces start on word boundaries

    def server_words(self) -> torch.Tensor:
        return self._cat(lambda e: e.server_words())

    def _scales(self, fn) -> torch.Tensor:
        out = torch.zeros(self.B, dtype=torch.float32, device=self.device)
        for rk in self.ranks:
            out[rk.gidx] = fn(rk.eng)                       # every piece holds the block's scale
        return out

    def worker_scales(self, i: int) -> torch.Tensor:
        return self._scales(lambda e: e.worker_scales(i))

    def server_scales(self) -> torch.Tensor:
        return self._scales(lambda e: e.server_scales())

    @property
    def step_count(self) -> int:
        counts = {rk.eng.step_count for rk in self.ranks}
        assert len(counts) == 1
        return counts.pop()


class _Gathered:
    """The concatenation of the ranks' parameter views: reads gather, copy_ scatters."""

    def __init__(self, owner: ShardedEngine, fn):
        self.owner, self.fn = owner, fn

    def _value(self) -> torch.Tensor:
        return torch.cat([self.fn(rk.eng) for rk in self.owner.ranks])

    def copy_(self, src: torch.Tensor):
        for rk in self.owner.ranks:
            self.fn(rk.eng).copy_(src[rk.shard.elem_lo:rk.shard.elem_hi])
        return self

    def numel(self) -> int:
        return self.owner.d

    def cpu(self):
        return self._value().cpu()

    def __getattr__(self, name):
        return getattr(self._value(), name)


class DistributedShard:
    """One rank of a torch.distributed group holding its element range of the layout; the
    exchange is an all-reduce of B doubles per cut-block call (skipped when no block is cut)."""

    def __init__(self, sizes: Sequence[int], M: int, mu: float, eta: float, rank: int, world: int,
                 group=None, granule: int = 4096, make_engine=_make_rank_engine, **engine_kw):
        self.sizes, self.rank, self.world, self.group = list(sizes), rank, world, group
        self.shard = shard_elements(self.sizes, world, rank, granule)
        self.any_cut = any(
            any(l != f for l, f in zip(s.local_sizes, s.full_sizes))
            for s in (shard_elements(self.sizes, world, r, granule) for r in range(world)))
        self.state = _RankState(self.shard, len(self.sizes), make_engine(self.shard, M, mu, eta, **engine_kw))
        self.eng = self.state.eng

    def _reduce_and_complete(self, who: int) -> None:
        if not self.any_cut:
            return
        import torch.distributed as dist
        total = self.state.sums_to_global(who)
        dist.all_reduce(total, op=dist.ReduceOp.SUM, group=self.group)
        if self.eng.B and any(l != f for l, f in zip(self.shard.local_sizes, self.shard.full_sizes)):
            self.state.complete(who, total)

    def worker_step_all(self, local_grads: torch.Tensor) -> None:
        """local_grads: [M, stride] for this rank's element range."""
        self.eng.worker_step_all(local_grads)
        for i in range(self.eng.M):
            self._reduce_and_complete(i)

    def server_step(self) -> None:
        self.eng.server_step_range(0, self.eng.B)
        self._reduce_and_complete(-1)
        self.eng.apply_update(0, self.eng.B)
