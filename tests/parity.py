"""Step-locked comparison of the CUDA path (through the C ABI) with the CPU oracle.

Protocol: both sides consume the same gradient buffer.  After each GPU call its packed words
go to the oracle as a hint; the oracle adopts a differing bit only where its own |p| is below
1e-6 x the block scale (either sign is a valid output of the compressor there) and lists the
element.  After adoption the packed words must be bit-identical.  Scales must agree to 1e-5
relative; momentum, residuals and parameters to 1e-5 of the block's largest magnitude.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from oracle import Oracle
from paper_1905_10936_b200.engine import EFEngine
from paper_1905_10936_b200.workloads import Workload

RTOL = 1e-5


def words_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


class BlockSample:
    """Maps a subset of blocks of a layout to a smaller, self-contained problem.  Blocks are
    independent in the method (every operation is per element or per block), so the oracle can
    be run on the subset alone."""

    def __init__(self, offsets: np.ndarray, blocks: Optional[Sequence[int]] = None):
        self.offsets = np.asarray(offsets, dtype=np.int64)
        B = len(self.offsets) - 1
        self.blocks = list(range(B)) if blocks is None else sorted(set(int(b) for b in blocks))
        self.full = blocks is None
        sizes = np.diff(self.offsets)
        woff = np.concatenate([[0], np.cumsum((sizes + 31) // 32)])
        self.sub_offsets = np.concatenate([[0], np.cumsum(sizes[self.blocks])])
        if self.full:
            self.elem_index = None
            self.word_index = None
        else:
            self.elem_index = torch.from_numpy(np.concatenate(
                [np.arange(self.offsets[b], self.offsets[b + 1]) for b in self.blocks]))
            self.word_index = torch.from_numpy(np.concatenate(
                [np.arange(woff[b], woff[b + 1]) for b in self.blocks]))
        self.block_index = torch.tensor(self.blocks, dtype=torch.int64)

    def elems(self, t: torch.Tensor) -> np.ndarray:
        if self.full:
            return t.cpu().numpy()
        return t[self.elem_index.to(t.device)].cpu().numpy()

    def words(self, t: torch.Tensor) -> np.ndarray:
        if self.full:
            return words_np(t)
        return words_np(t[self.word_index.to(t.device)])

    def scales(self, t: torch.Tensor) -> np.ndarray:
        if self.full:
            return t.cpu().numpy()
        return t[self.block_index.to(t.device)].cpu().numpy()


def assert_blockwise_close(got: np.ndarray, ref: np.ndarray, sub_offsets: np.ndarray, what: str):
    """max_j |got - ref| <= RTOL * max_j |ref| within every block."""
    diff = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    mx_d = np.maximum.reduceat(diff, sub_offsets[:-1])
    mx_r = np.maximum.reduceat(np.abs(ref).astype(np.float64), sub_offsets[:-1])
    bad = np.nonzero(mx_d > RTOL * mx_r)[0]
    assert bad.size == 0, (f"{what}: {bad.size} blocks out of tolerance; first block {bad[0]}: "
                           f"err {mx_d[bad[0]]:.3e} vs max|ref| {mx_r[bad[0]]:.3e}")


def assert_scales_close(got: np.ndarray, ref: np.ndarray, what: str):
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    assert np.all(err <= RTOL * np.abs(ref)), f"{what}: scale mismatch, max rel err " \
        f"{(err / np.maximum(np.abs(ref), 1e-300)).max():.3e}"


def run_parity(w: Workload, steps: Optional[int] = None, blocks: Optional[Sequence[int]] = None,
               grads: Optional[List[List[torch.Tensor]]] = None, check_every_step: bool = True,
               device: str = "cuda", scale_mode: str = "auto", batched: bool = False,
               etas: Optional[Sequence[float]] = None, weight_decay: float = 0.0,
               x0: Optional[torch.Tensor] = None, diagnostics: bool = False):
    """Runs `steps` iterations on both sides; returns (engine, oracle, stats)."""
    steps = w.steps if steps is None else steps
    eta0 = w.eta if etas is None else etas[0]
    eng = EFEngine(w.offsets, w.M, w.mu, eta0, scale_mode=scale_mode, weight_decay=weight_decay > 0,
                   diagnostics=diagnostics)
    smp = BlockSample(w.offsets, blocks)
    orc = Oracle(smp.sub_offsets, w.M, w.mu, eta0)
    if weight_decay > 0:
        eng.set_weight_decay(weight_decay)
        orc.set_weight_decay(weight_decay)
    if x0 is not None:
        eng.params().copy_(x0.to(device))
        orc.x[:] = smp.elems(x0.to(device))
    es = w.element_scales(device)
    gbuf = torch.empty(w.d, dtype=torch.float32, device=device)
    # batched mode: all M gradients in one [M, stride] tensor, one ef_worker_step_all per step
    stride = (w.d + 3) // 4 * 4
    gall = torch.zeros(w.M, stride, dtype=torch.float32, device=device) if batched else None
    stats = {"adopted": 0, "scale_bit_mismatch": 0, "scales_compared": 0, "adopted_list": []}
    for t in range(steps):
        if etas is not None and t > 0:
            eng.set_eta(etas[t])
            orc.set_eta(etas[t])
        if batched:
            for i in range(w.M):
                if grads is not None:
                    gall[i, :w.d].copy_(grads[t][i])
                else:
                    w.draw_grad(t, i, device, es, out=gall[i, :w.d])
            eng.worker_step_all(gall)
        for i in range(w.M):
            if batched:
                g = gall[i, :w.d]
            else:
                g = grads[t][i].to(device) if grads is not None else w.draw_grad(t, i, device, es, out=gbuf)
                eng.worker_step(i, g)
            gw = smp.words(eng.worker_words(i))
            ad = orc.worker_step(i, smp.elems(g), hint=gw)
            stats["adopted"] += len(ad)
            stats["adopted_list"] += [("worker", t, i, int(j)) for j in ad]
            assert np.array_equal(orc.words(i), gw), \
                f"worker {i} step {t}: packed words differ outside the tie zone"
            gs = smp.scales(eng.worker_scales(i))
            assert_scales_close(gs, orc.scales(i), f"worker {i} step {t}")
            stats["scale_bit_mismatch"] += int((gs != orc.scales(i)).sum())
            stats["scales_compared"] += gs.size
            if diagnostics:
                # ||p||_1 is the compressor's own fp64 sum (1e-11); the three diagnostic sums
                # combine each lane's four elements in fp32 first: <= 4 * 2^-24 relative
                gd = eng.worker_diagnostics(i)[smp.block_index.to(device)].cpu().numpy()
                od = orc.diagnostics(i)
                tol = np.array([1e-11, 1e-6, 1e-6, 1e-6])
                assert np.all(np.abs(gd - od) <= tol * np.abs(od)), \
                    f"worker {i} step {t}: diagnostics differ, max rel " \
                    f"{(np.abs(gd - od) / np.maximum(np.abs(od), 1e-300)).max():.3e}"
        eng.server_step()
        gw = smp.words(eng.server_words())
        ad = orc.server_step(hint=gw)
        stats["adopted"] += len(ad)
        stats["adopted_list"] += [("server", t, -1, int(j)) for j in ad]
        assert np.array_equal(orc.words(-1), gw), \
            f"server step {t}: packed words differ outside the tie zone"
        gs = smp.scales(eng.server_scales())
        assert_scales_close(gs, orc.scales(-1), f"server step {t}")
        stats["scale_bit_mismatch"] += int((gs != orc.scales(-1)).sum())
        stats["scales_compared"] += gs.size
        if check_every_step or t == steps - 1:
            compare_state(eng, orc, smp, f"after step {t}")
    assert eng.step_count == steps == orc.t
    if weight_decay > 0:
        assert_blockwise_close(smp.elems(eng.decay_momentum()), orc.decay_momentum, smp.sub_offsets,
                               "decay momentum")
    return eng, orc, stats


def compare_state(eng: EFEngine, orc: Oracle, smp: BlockSample, when: str):
    so = smp.sub_offsets
    assert_blockwise_close(smp.elems(eng.params()), orc.x, so, f"x {when}")
    assert_blockwise_close(smp.elems(eng.residual(-1)), orc.residual(-1), so, f"server residual {when}")
    for i in range(eng.M):
        assert_blockwise_close(smp.elems(eng.momentum(i)), orc.momentum(i), so, f"m[{i}] {when}")
        assert_blockwise_close(smp.elems(eng.residual(i)), orc.residual(i), so, f"e[{i}] {when}")
