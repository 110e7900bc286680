"""Pins for the oracle of the two comparison compressors: signum with majority vote and top-k.

None of these re-types the oracle's loops: expectations come from a hand-worked table, exact
rational arithmetic, numpy evaluating the textbook definition sign(sum_i sign(.)), invariants of
the method (scale invariance, unit steps, message sizes of Table 1), Definition 1's inequality
with delta = k/d, and brute force over all k-subsets on tiny inputs.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import SignumOracle, topk_compress

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "signum_vote_hand_case.txt")


def _cases():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, _, rest = line.partition(" ")
        if key == "case":
            cur = {"name": rest, "grad": {}, "rows": []}
            cases.append(cur)
        elif key in ("d", "M"):
            cur[key] = int(rest)
        elif key in ("mu", "eta"):
            cur[key] = float(rest)
        elif key == "offsets":
            cur["offsets"] = [int(v) for v in rest.split()]
        elif key == "grad":
            f = rest.split()
            cur["grad"][(int(f[0]), int(f[1]))] = np.array([float(v) for v in f[2:]], dtype=np.float32)
        else:
            head, *cols = [c.split() for c in rest.split("|")]
            cur["rows"].append((key, [int(v) for v in head], cols))
    return cases


def _unpack(words, offsets):
    out = []
    woff = 0
    for b in range(len(offsets) - 1):
        n = offsets[b + 1] - offsets[b]
        for k in range(n):
            out.append((int(words[woff + k // 32]) >> (k % 32)) & 1)
        woff += (n + 31) // 32
    return out


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"])
def test_hand_worked_table(case):
    o = SignumOracle(case["offsets"], case["M"], case["mu"], case["eta"])
    for who, head, cols in case["rows"]:
        if who == "worker":
            t, i = head
            o.worker_step(i, case["grad"][(t, i)])
            assert o.momentum(i).tolist() == [float(v) for v in cols[0]]
            assert _unpack(o.words(i), case["offsets"]) == [int(v) for v in cols[1]]
            assert o.words(i).tolist() == [int(v) for v in cols[2]]
        else:
            o.server_step()
            assert _unpack(o.words(-1), case["offsets"]) == [int(v) for v in cols[0]]
            assert o.words(-1).tolist() == [int(v) for v in cols[1]]
            assert o.x.tolist() == [float(v) for v in cols[2]]


def _dyadic(rng, n, bits=6):
    return (rng.integers(-(1 << bits), (1 << bits) + 1, size=n) / float(1 << 3)).astype(np.float32)


@pytest.mark.parametrize("M", [1, 3, 4, 7])
def test_against_exact_rationals_and_the_textbook_vote(M):
    """Momentum recurrence in exact rationals (dyadic inputs, mu = 1/2: binary32 is exact), vote
    as numpy's sign of the sum of signs; odd M can never tie (Section 4.2)."""
    rng = np.random.default_rng(10 + M)
    sizes = [3, 32, 33, 70]
    off = np.concatenate([[0], np.cumsum(sizes)])
    d, steps, mu, eta = int(off[-1]), 4, 0.5, 0.125
    o = SignumOracle(off, M, mu, eta)
    m = [[Fraction(0)] * d for _ in range(M)]
    x = [Fraction(0)] * d
    for t in range(steps):
        signs = np.zeros((M, d), dtype=np.int64)
        for i in range(M):
            g = _dyadic(rng, d)
            o.worker_step(i, g)
            m[i] = [Fraction(mu) * a + Fraction(float(b)) for a, b in zip(m[i], g)]
            signs[i] = [-1 if v < 0 else 1 for v in m[i]]
            assert [Fraction(float(v)) for v in o.momentum(i)] == m[i]
            assert _unpack(o.words(i), off) == [int(s < 0) for s in signs[i]]
        o.server_step()
        total = signs.sum(axis=0)
        if M % 2 == 1:
            assert (total != 0).all()
        vote = np.where(np.sign(total) < 0, -1, 1)         # tie -> +1
        assert _unpack(o.words(-1), off) == [int(v < 0) for v in vote]
        x = [a - Fraction(eta) * int(v) for a, v in zip(x, vote)]
        assert [Fraction(float(v)) for v in o.x] == x
        # padding bits of every block's last word stay zero
        woff = np.concatenate([[0], np.cumsum([(s + 31) // 32 for s in sizes])])
        for b, s in enumerate(sizes):
            if s % 32:
                for wv in (o.words(-1), o.words(0)):
                    assert int(wv[woff[b + 1] - 1]) >> (s % 32) == 0


def test_single_worker_vote_is_its_own_sign_and_steps_are_unit():
    rng = np.random.default_rng(2)
    d, eta = 100, 2.0 ** -4
    o = SignumOracle([0, 40, d], 1, 0.9, eta)
    for t in range(7):
        o.worker_step(0, rng.standard_normal(d).astype(np.float32))
        o.server_step()
        assert np.array_equal(o.words(-1), o.words(0))
    steps = o.x / eta                                       # every coordinate moved by +-eta per step
    assert np.all(np.abs(steps) <= 7) and np.all((steps.astype(np.int64) - 7) % 2 == 0)
    assert np.array_equal(steps, np.round(steps))


def test_only_the_direction_of_the_gradients_matters():
    """Scaling every gradient by a positive constant (a power of two, so binary32 scales
    exactly) changes no message and no parameter: no magnitude enters the method."""
    rng = np.random.default_rng(3)
    off = [0, 31, 64, 200]
    a, b = SignumOracle(off, 4, 0.5, 0.1), SignumOracle(off, 4, 0.5, 0.1)
    for t in range(5):
        for i in range(4):
            g = rng.standard_normal(200).astype(np.float32)
            a.worker_step(i, g); b.worker_step(i, g * np.float32(1024.0))
            assert np.array_equal(a.words(i), b.words(i))
        a.server_step(); b.server_step()
        assert np.array_equal(a.words(-1), b.words(-1)) and np.array_equal(a.x, b.x)


def test_message_sizes_of_table_1():
    """Table 1: 2Md bits per iteration (d bits up, d bits down, per worker) when every block
    is a multiple of 32 elements; no scales travel."""
    sizes = [64, 96, 32 * 7]
    off = np.concatenate([[0], np.cumsum(sizes)])
    o = SignumOracle(off, 5, 0.9, 0.1)
    assert 32 * o.W == off[-1]
    assert 2 * o.M * 32 * o.W == 2 * 5 * off[-1]


def test_call_order_is_enforced():
    o = SignumOracle([0, 8], 2, 0.9, 0.1)
    g = np.ones(8, dtype=np.float32)
    with pytest.raises(RuntimeError):
        o.server_step()
    o.worker_step(0, g)
    with pytest.raises(RuntimeError):
        o.worker_step(0, g)
    with pytest.raises(ValueError):
        SignumOracle([0, 8], 2, 1.0, 0.1)


# ------------------------------------------------------------------ top-k
def test_topk_small_examples():
    idx, val, r = topk_compress(np.array([1, -5, 3, 5, 0, -2], dtype=np.float32), 3)
    assert idx.tolist() == [1, 2, 3] and val.tolist() == [-5.0, 3.0, 5.0]
    assert r.tolist() == [1.0, 0.0, 0.0, 0.0, 0.0, -2.0]
    # equal magnitudes: the lower index wins (a reading); +0 and -0 tie as well
    idx, val, _ = topk_compress(np.array([2, -2, 2, -2], dtype=np.float32), 2)
    assert idx.tolist() == [0, 1] and val.tolist() == [2.0, -2.0]
    idx, _, _ = topk_compress(np.array([0.0, -0.0, 0.0], dtype=np.float32), 2)
    assert idx.tolist() == [0, 1]
    v = np.array([3, -1, 4, 1, -5, 9, 2, -6], dtype=np.float32)
    idx, val, r = topk_compress(v, 8)                      # k = d: the identity, residual 0
    assert idx.tolist() == list(range(8)) and np.array_equal(val, v) and not r.any()
    idx, val, _ = topk_compress(v, 1)                      # k = 1: the entry of largest magnitude
    assert idx.tolist() == [int(np.argmax(np.abs(v)))] and val.tolist() == [9.0]
    for bad_k in (0, 9):
        with pytest.raises(ValueError):
            topk_compress(v, bad_k)


@pytest.mark.parametrize("n,k", [(6, 1), (7, 3), (9, 4), (10, 5), (10, 9)])
def test_topk_minimises_the_residual_over_all_k_subsets(n, k):
    """Brute force: among all ways to keep k coordinates, top-k leaves the smallest residual
    (that is what makes it a delta-approximate compressor with delta = k/d, Definition 1)."""
    rng = np.random.default_rng(100 * n + k)
    v = rng.standard_normal(n).astype(np.float32)
    idx, val, r = topk_compress(v, k)
    best = min(float(np.sum(np.delete(v.astype(np.float64), list(c)) ** 2))
               for c in itertools.combinations(range(n), k))
    assert abs(float(np.sum(r.astype(np.float64) ** 2)) - best) <= 1e-12


@pytest.mark.parametrize("law", ["normal", "laplace", "heavy"])
def test_topk_invariants_and_definition_1(law):
    rng = np.random.default_rng(5)
    n = 5000
    v = {"normal": rng.standard_normal(n), "laplace": rng.laplace(size=n),
         "heavy": rng.standard_cauchy(n)}[law].astype(np.float32)
    v[::97] = 0.0
    v[1::89] = v[0]                                         # repeated magnitudes
    for k in (1, 17, n // 10, n - 1):
        idx, val, r = topk_compress(v, k)
        assert len(idx) == k and np.all(np.diff(idx) > 0)   # exactly k entries, increasing
        assert np.array_equal(val, v[idx])
        kept = np.zeros(n, dtype=bool); kept[idx] = True
        assert np.abs(v[kept]).min() >= np.abs(v[~kept]).max()
        assert not r[kept].any() and np.array_equal(r[~kept], v[~kept])    # e = v - C(v)
        # ties at the threshold go to the lowest indices
        thr = np.abs(v[kept]).min()
        tied = np.nonzero(np.abs(v) == thr)[0]
        n_tied_kept = int(kept[tied].sum())
        assert kept[tied[:n_tied_kept]].all()
        # Definition 1 with delta = k/d
        v64 = v.astype(np.float64)
        assert np.sum(r.astype(np.float64) ** 2) <= (1 - k / n) * np.sum(v64 ** 2) * (1 + 1e-12)
