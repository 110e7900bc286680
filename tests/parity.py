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
from oracle_pool import OraclePool, blockwise_check
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


class _SingleOracle:
    """The oracle in this process, on the blocks the sample names."""

    def __init__(self, smp: "BlockSample", M, mu, eta, diagnostics):
        self.smp = smp
        self.orc = Oracle(smp.sub_offsets, M, mu, eta, diagnostics=diagnostics)

    def _step(self, i, gw, ad):
        neq = np.nonzero(self.orc.words(i) != gw)[0]
        return ad, (int(neq[0]) if neq.size else -1), self.orc.scales(i)

    def worker_step(self, i, g: torch.Tensor, words: torch.Tensor):
        gw = self.smp.words(words)
        return self._step(i, gw, self.orc.worker_step(i, self.smp.elems(g), hint=gw))

    def server_step(self, words: torch.Tensor):
        gw = self.smp.words(words)
        return self._step(-1, gw, self.orc.server_step(hint=gw))

    def set_eta(self, eta):
        self.orc.set_eta(eta)

    def set_weight_decay(self, lam):
        self.orc.set_weight_decay(lam)

    def set_x(self, x0: torch.Tensor):
        self.orc.x[:] = self.smp.elems(x0)

    def compare(self, kind, i, got: torch.Tensor):
        ref = {"x": lambda: self.orc.x, "m": lambda: self.orc.momentum(i),
               "e": lambda: self.orc.residual(i), "mt": lambda: self.orc.decay_momentum}[kind]()
        return blockwise_check(self.smp.elems(got), ref, self.smp.sub_offsets)

    def diagnostics(self, i):
        return self.orc.diagnostics(i)

    @property
    def t(self):
        return self.orc.t

    def close(self):
        self.orc.close()


class _PooledOracle:
    """The oracle on the whole layout, spread over processes by block range (oracle_pool.py)."""

    def __init__(self, smp: "BlockSample", M, mu, eta, nproc):
        assert smp.full, "the process pool follows the whole vector"
        self.pool = OraclePool(smp.offsets, M, mu, eta, nproc)
        self.orc = None
        self._views = [torch.from_numpy(a) for a in (self.pool.grad, self.pool.hint.view(np.int32),
                                                     self.pool.state)]
        # page-lock the shared buffers so device-to-host copies run at full PCIe rate; harmless
        # if the driver refuses
        self._registered = []
        try:
            rt = torch.cuda.cudart()
            for v in self._views:
                if int(rt.cudaHostRegister(v.data_ptr(), v.numel() * v.element_size(), 0)) == 0:
                    self._registered.append(v.data_ptr())
        except Exception:
            pass

    def worker_step(self, i, g, words):
        self._views[0].copy_(g)
        self._views[1].copy_(words)
        return self.pool.worker_step(i)

    def server_step(self, words):
        self._views[1].copy_(words)
        return self.pool.server_step()

    def set_eta(self, eta):
        self.pool.set_eta(eta)

    def set_weight_decay(self, lam):
        self.pool.set_weight_decay(lam)

    def set_x(self, x0):
        self._views[2].copy_(x0)
        self.pool.set_x_from_state()

    def compare(self, kind, i, got):
        self._views[2].copy_(got)
        return self.pool.compare(kind, i)

    @property
    def t(self):
        return self.pool.t

    def close(self):
        try:
            rt = torch.cuda.cudart()
            for ptr in self._registered:
                rt.cudaHostUnregister(ptr)
        except Exception:
            pass
        self._registered, self._views = [], []
        self.pool.close()


def _check_state(side, kind, i, got, what, stats, clean):
    """State vector against the oracle: within RTOL of the block's largest magnitude; and, as
    long as no tie-zone bit was adopted and every scale agreed bit for bit, the same binary32
    number in every element (both sides evaluate Algorithm 4 in the same operation order; +0 and
    -0 count as the same number)."""
    bad, mism = side.compare(kind, i, got)
    assert not bad, (f"{what}: {len(bad)} blocks out of tolerance; first block {bad[0][0]}: "
                     f"err {bad[0][1]:.3e} vs max|ref| {bad[0][2]:.3e}")
    stats["state_value_mismatch"] += mism
    stats["state_elements_compared"] += got.numel()
    if clean:
        assert mism == 0, f"{what}: {mism} elements differ from the oracle's value"


def assert_scales_close(got: np.ndarray, ref: np.ndarray, what: str):
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    assert np.all(err <= RTOL * np.abs(ref)), f"{what}: scale mismatch, max rel err " \
        f"{(err / np.maximum(np.abs(ref), 1e-300)).max():.3e}"


def run_parity(w: Workload, steps: Optional[int] = None, blocks: Optional[Sequence[int]] = None,
               grads: Optional[List[List[torch.Tensor]]] = None, check_every_step: bool = True,
               device: str = "cuda", scale_mode: str = "auto", batched: bool = False,
               etas: Optional[Sequence[float]] = None, weight_decay: float = 0.0,
               x0: Optional[torch.Tensor] = None, diagnostics: bool = False,
               oracle_procs: int = 0, engine_factory=None):
    """Runs `steps` iterations on both sides; returns (engine, oracle side, stats).

    oracle_procs > 1 spreads the oracle over that many processes by block range (whole vector
    only); otherwise one oracle instance runs in this process on the sampled blocks.
    engine_factory(offsets, M, mu, eta, **kw) may supply another object with EFEngine's methods
    (used to drive the same protocol through other entry points)."""
    steps = w.steps if steps is None else steps
    eta0 = w.eta if etas is None else etas[0]
    make = engine_factory or EFEngine
    eng = make(w.offsets, w.M, w.mu, eta0, scale_mode=scale_mode, weight_decay=weight_decay > 0,
               diagnostics=diagnostics)
    smp = BlockSample(w.offsets, blocks)
    if oracle_procs > 1:
        assert not diagnostics
        side = _PooledOracle(smp, w.M, w.mu, eta0, oracle_procs)
    else:
        side = _SingleOracle(smp, w.M, w.mu, eta0, diagnostics)
    stats = {"adopted": 0, "scale_bit_mismatch": 0, "scales_compared": 0, "adopted_list": [],
             "state_value_mismatch": 0, "state_elements_compared": 0}
    try:
        _run(w, eng, side, smp, stats, steps, grads, check_every_step, device, batched, etas,
             weight_decay, x0, diagnostics)
    except BaseException:
        side.close()
        raise
    if oracle_procs > 1:
        side.close()
    return eng, side.orc, stats


def _run(w, eng, side, smp, stats, steps, grads, check_every_step, device, batched, etas,
         weight_decay, x0, diagnostics):
    if weight_decay > 0:
        eng.set_weight_decay(weight_decay)
        side.set_weight_decay(weight_decay)
    if x0 is not None:
        eng.params().copy_(x0.to(device))
        side.set_x(x0.to(device))
    es = w.element_scales(device)
    gbuf = torch.empty(w.d, dtype=torch.float32, device=device)
    # batched mode: all M gradients in one [M, stride] tensor, one ef_worker_step_all per step
    stride = (w.d + 3) // 4 * 4
    gall = torch.zeros(w.M, stride, dtype=torch.float32, device=device) if batched else None

    def after_call(who, t, i, res, scales_t):
        ad, first_diff, ref_scales = res
        stats["adopted"] += len(ad)
        stats["adopted_list"] += [(who, t, i, int(j)) for j in ad]
        assert first_diff < 0, \
            f"{who} {i} step {t}: packed words differ outside the tie zone (first at word {first_diff})"
        gs = smp.scales(scales_t)
        assert_scales_close(gs, ref_scales, f"{who} {i} step {t}")
        stats["scale_bit_mismatch"] += int((gs != ref_scales).sum())
        stats["scales_compared"] += gs.size

    for t in range(steps):
        if etas is not None and t > 0:
            eng.set_eta(etas[t])
            side.set_eta(etas[t])
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
            after_call("worker", t, i, side.worker_step(i, g, eng.worker_words(i)), eng.worker_scales(i))
            if diagnostics:
                # ||p||_1 is the compressor's own fp64 sum (1e-11); the three diagnostic sums
                # combine each lane's four elements in fp32 first: <= 4 * 2^-24 relative
                gd = eng.worker_diagnostics(i)[smp.block_index.to(device)].cpu().numpy()
                od = side.diagnostics(i)
                tol = np.array([1e-11, 1e-6, 1e-6, 1e-6])
                assert np.all(np.abs(gd - od) <= tol * np.abs(od)), \
                    f"worker {i} step {t}: diagnostics differ, max rel " \
                    f"{(np.abs(gd - od) / np.maximum(np.abs(od), 1e-300)).max():.3e}"
        eng.server_step()
        after_call("server", t, -1, side.server_step(eng.server_words()), eng.server_scales())
        if check_every_step or t == steps - 1:
            compare_state(eng, side, stats, f"after step {t}")
    assert eng.step_count == steps == side.t
    if weight_decay > 0:
        clean = stats["adopted"] == 0 and stats["scale_bit_mismatch"] == 0
        _check_state(side, "mt", -1, eng.decay_momentum(), "decay momentum", stats, clean)


def compare_state(eng, side, stats, when: str):
    clean = stats["adopted"] == 0 and stats["scale_bit_mismatch"] == 0
    _check_state(side, "x", -1, eng.params(), f"x {when}", stats, clean)
    _check_state(side, "e", -1, eng.residual(-1), f"server residual {when}", stats, clean)
    for i in range(eng.M):
        _check_state(side, "m", i, eng.momentum(i), f"m[{i}] {when}", stats, clean)
        _check_state(side, "e", i, eng.residual(i), f"e[{i}] {when}", stats, clean)
