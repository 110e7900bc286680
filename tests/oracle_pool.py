"""Several untouched, single-threaded oracle instances on disjoint block ranges, one per process.

Every operation of the method is per element or per block (Algorithm 4; the blockwise
compressor of Section 3.2 never looks across blocks), so the oracle's result on the whole
vector is the concatenation of its results on block ranges.  That is all this module uses: each
child process owns a contiguous range of whole blocks and runs the plain `oracle.Oracle` on it.
The oracle itself is neither threaded nor changed.  It lets the full-size layouts (2^28 and
3.5e8 parameters) be followed element by element within the time a test may take.

The parent and the children exchange vectors through three shared buffers (one gradient, one
set of packed words, one state vector: files mapped by every process, in /dev/shm when it has
the room); small results travel over pipes.  This module
imports no torch and no CUDA: the children are spawned, not forked, and never touch a device.
"""
from __future__ import annotations

import multiprocessing as mp
import os
import shutil
import tempfile
from typing import List, Optional, Sequence, Tuple

import numpy as np

RTOL = 1e-5


def split_blocks(sizes: Sequence[int], parts: int) -> List[Tuple[int, int]]:
    """Cuts B blocks into at most `parts` contiguous non-empty ranges of similar element count."""
    sizes = np.asarray(sizes, dtype=np.int64)
    B = len(sizes)
    parts = max(1, min(parts, B))
    cum = np.concatenate([[0], np.cumsum(sizes)])
    cuts = [0]
    for r in range(1, parts):
        b = int(np.searchsorted(cum, cum[-1] * r / parts, side="left"))
        b = min(max(b, cuts[-1] + 1), B - (parts - r))
        cuts.append(b)
    cuts.append(B)
    return [(cuts[k], cuts[k + 1]) for k in range(parts) if cuts[k + 1] > cuts[k]]


def blockwise_check(got: np.ndarray, ref: np.ndarray, sub_offsets: np.ndarray):
    """Per block: max |got - ref| against RTOL * max |ref|.  Returns (bad, mismatch):
    bad = [(block, err, max_ref)] for the blocks out of tolerance, mismatch = number of
    elements that are not the same binary32 number (+0 and -0 are the same number: the method
    reads sign(+-0) = +1 and never divides by a state value, so the two are interchangeable)."""
    diff = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    mx_d = np.maximum.reduceat(diff, sub_offsets[:-1])
    mx_r = np.maximum.reduceat(np.abs(ref).astype(np.float64), sub_offsets[:-1])
    bad = [(int(b), float(mx_d[b]), float(mx_r[b])) for b in np.nonzero(mx_d > RTOL * mx_r)[0]]
    mism = int(np.count_nonzero(got != ref))
    return bad, mism


def _attach(path: str, n: int, dtype):
    return np.memmap(path, dtype=dtype, mode="r+", shape=(max(n, 1),))[:n]


def _shared_dir(nbytes: int) -> str:
    """A directory for the shared buffers: memory-backed /dev/shm when it has the room, else the
    ordinary temporary directory (slower, but it cannot run out of space under a write)."""
    for base in ("/dev/shm", tempfile.gettempdir()):
        try:
            st = os.statvfs(base)
            if st.f_bavail * st.f_frsize > nbytes + (64 << 20):
                return tempfile.mkdtemp(prefix="oracle_pool_", dir=base)
        except OSError:
            pass
    return tempfile.mkdtemp(prefix="oracle_pool_")


def _child(conn, names, d, W, offsets, woffsets, b0, b1, M, mu, eta):
    from oracle import Oracle
    g = _attach(names[0], d, np.float32)
    hint = _attach(names[1], W, np.uint32)
    buf = _attach(names[2], d, np.float32)
    lo, hi = int(offsets[b0]), int(offsets[b1])
    wlo, whi = int(woffsets[b0]), int(woffsets[b1])
    sub = np.ascontiguousarray(offsets[b0:b1 + 1] - offsets[b0])
    orc = Oracle(sub, M, mu, eta)
    try:
        while True:
            cmd = conn.recv()
            op = cmd[0]
            if op == "exit":
                break
            if op in ("worker", "server"):
                i = cmd[1] if op == "worker" else -1
                h = hint[wlo:whi]
                ad = orc.worker_step(i, g[lo:hi], hint=h) if op == "worker" else orc.server_step(hint=h)
                mine = orc.words(i)
                neq = np.nonzero(mine != h)[0]
                first = int(neq[0]) + wlo if neq.size else -1
                conn.send((ad + lo, first, orc.scales(i).copy()))
            elif op == "cmp":
                kind, i = cmd[1], cmd[2]
                ref = {"x": lambda: orc.x, "m": lambda: orc.momentum(i),
                       "e": lambda: orc.residual(i), "mt": lambda: orc.decay_momentum}[kind]()
                bad, mism = blockwise_check(buf[lo:hi], ref, sub)
                conn.send(([(b + b0, e, r) for b, e, r in bad], mism))
            elif op == "set_eta":
                orc.set_eta(cmd[1]); conn.send(None)
            elif op == "set_weight_decay":
                orc.set_weight_decay(cmd[1]); conn.send(None)
            elif op == "set_x":
                orc.x[:] = buf[lo:hi]; conn.send(None)
            elif op == "t":
                conn.send(orc.t)
            else:
                conn.send(RuntimeError(f"unknown command {op}"))
    finally:
        orc.close()
        del g, hint, buf


class OraclePool:
    """The oracle on a whole layout, computed by `nproc` processes on disjoint block ranges.

    The caller fills `grad` (d floats), `hint` (W packed words of the other implementation) and
    `state` (d floats) -- numpy views of the shared buffers -- and then calls the step or
    comparison method; all children work at the same time and the method gathers their answers.
    """

    def __init__(self, offsets, M: int, mu: float, eta: float, nproc: Optional[int] = None):
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        sizes = np.diff(self.offsets)
        self.B, self.d, self.M = len(sizes), int(self.offsets[-1]), int(M)
        self.woffsets = np.concatenate([[0], np.cumsum((sizes + 31) // 32)]).astype(np.int64)
        self.W = int(self.woffsets[-1])
        nproc = nproc or min(os.cpu_count() or 1, 16)
        self.ranges = split_blocks(sizes, nproc)
        self._dir = _shared_dir(4 * (2 * self.d + self.W))
        names = [os.path.join(self._dir, n) for n in ("grad", "hint", "state")]
        for path, n in zip(names, (self.d, self.W, self.d)):
            with open(path, "wb") as f:
                f.truncate(4 * max(n, 1))
        self.grad = _attach(names[0], self.d, np.float32)
        self.hint = _attach(names[1], self.W, np.uint32)
        self.state = _attach(names[2], self.d, np.float32)
        ctx = mp.get_context("spawn")
        self._procs, self._conns = [], []
        for (b0, b1) in self.ranges:
            parent, child = ctx.Pipe()
            p = ctx.Process(target=_child, args=(child, names, self.d, self.W, self.offsets,
                                                 self.woffsets, b0, b1, self.M, float(mu), float(eta)),
                            daemon=True)
            p.start()
            child.close()
            self._procs.append(p)
            self._conns.append(parent)

    # ---- plumbing ---------------------------------------------------------------------------
    def _all(self, *cmd):
        for c in self._conns:
            c.send(cmd)
        out = [c.recv() for c in self._conns]
        for o in out:
            if isinstance(o, Exception):
                raise o
        return out

    def close(self):
        if getattr(self, "_conns", None):
            for c in self._conns:
                try:
                    c.send(("exit",))
                except Exception:
                    pass
            for p in self._procs:
                p.join(timeout=30)
                if p.is_alive():
                    p.terminate()          # the exact child this pool started
            self._conns, self._procs = [], []
            self.grad = self.hint = self.state = None
            shutil.rmtree(self._dir, ignore_errors=True)

    def __del__(self):
        self.close()

    # ---- steps: the caller has filled self.grad / self.hint ----------------------------------
    def _gather_step(self, res):
        adopted = np.concatenate([r[0] for r in res]) if res else np.zeros(0, np.int64)
        firsts = [r[1] for r in res if r[1] >= 0]
        scales = np.concatenate([r[2] for r in res])
        return adopted, (min(firsts) if firsts else -1), scales

    def worker_step(self, i: int):
        """Returns (adopted flat indices, first packed word that differs from the hint after
        adoption or -1, the oracle's B scales)."""
        return self._gather_step(self._all("worker", int(i)))

    def server_step(self):
        return self._gather_step(self._all("server"))

    def set_eta(self, eta: float):
        self._all("set_eta", float(eta))

    def set_weight_decay(self, lam: float):
        self._all("set_weight_decay", float(lam))

    def set_x_from_state(self):
        """x <- the vector in self.state."""
        self._all("set_x")

    @property
    def t(self) -> int:
        ts = self._all("t")
        assert len(set(ts)) == 1
        return ts[0]

    # ---- comparison: the caller has filled self.state with the other side's vector -----------
    def compare(self, kind: str, i: int = -1):
        """kind: "x", "m", "e" (i = -1: server residual) or "mt".  Returns (bad blocks, number of
        elements that differ in value)."""
        res = self._all("cmp", kind, int(i))
        bad = [b for r in res for b in r[0]]
        return bad, sum(r[1] for r in res)
