"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the passage it takes its expectation from.  None of them re-types the
oracle's loops: expectations come from hand-worked tables (tests/golden), exact rational
arithmetic, closed forms, identities, or textbook routines the method reduces to.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import Oracle
from exact_alg4 import ExactAlg4

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- helpers
def decode(words, scales, offsets):
    """Independent decoder of the wire format: bit k of a block's words, LSB first,
    1 = negative; value = -+scale.  Uses numpy's unpackbits, not the oracle."""
    offsets = np.asarray(offsets)
    out = np.empty(int(offsets[-1]), dtype=np.float64)
    w0 = 0
    for b in range(len(offsets) - 1):
        db = int(offsets[b + 1] - offsets[b])
        nw = (db + 31) // 32
        bits = np.unpackbits(np.asarray(words[w0:w0 + nw], dtype="<u4").view(np.uint8),
                             bitorder="little")
        assert not bits[db:].any(), "padding bits must be zero"
        out[offsets[b]:offsets[b + 1]] = np.where(bits[:db] == 1, -1.0, 1.0) * float(scales[b])
        w0 += nw
    assert w0 == len(words)
    return out


def run_steps(o, grads_per_step):
    for grads in grads_per_step:
        for i, g in enumerate(grads):
            o.worker_step(i, g)
        o.server_step()


def parse_hand_case(path):
    cfg, grads, rows = {}, {}, []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(None, 1)
        if key in ("d", "M", "steps"):
            cfg[key] = int(rest)
        elif key in ("mu", "eta"):
            cfg[key] = float(rest)
        elif key == "offsets":
            cfg[key] = [int(t) for t in rest.split()]
        elif key == "grad":
            t = rest.split()
            grads[(int(t[0]), int(t[1]))] = [float(v) for v in t[2:]]
        elif key in ("worker", "server"):
            head, *cols = [c.strip() for c in rest.split("|")]
            rows.append((key, [int(v) for v in head.split()],
                         [[float(v) for v in c.split()] for c in cols]))
    return cfg, grads, rows


# ---------------------------------------------------------------- P1: hand-worked Algorithm 4
def test_hand_case_e1_matches_oracle():
    cfg, grads, rows = parse_hand_case(os.path.join(GOLDEN, "alg4_hand_case_e1.txt"))
    o = Oracle(cfg["offsets"], cfg["M"], cfg["mu"], cfg["eta"])
    for kind, head, cols in rows:
        if kind == "worker":
            t, i = head
            m, p, scales, bits, words, resid = cols
            o.worker_step(i, np.array(grads[(t, i)], dtype=np.float32))
            assert o.momentum(i).tolist() == m
            assert o.last_p.tolist() == p
            assert o.scales(i).tolist() == scales
            assert o.words(i).tolist() == [int(w) for w in words]
            assert o.residual(i).tolist() == resid
            # the bit column and the word column of the fixture agree with the stated layout
            off = cfg["offsets"]
            for b in range(len(off) - 1):
                blk = bits[off[b]:off[b + 1]]
                assert int(words[b]) == sum(int(v) << k for k, v in enumerate(blk))
        else:
            (t,) = head
            p, scales, bits, words, resid, x = cols
            o.server_step()
            assert o.last_p.tolist() == p
            assert o.scales(-1).tolist() == scales
            assert o.words(-1).tolist() == [int(w) for w in words]
            assert o.residual(-1).tolist() == resid
            assert o.x.tolist() == x
            assert o.t == t + 1


def test_hand_case_e1_matches_exact_rationals():
    """The fixture itself is checked against exact rational arithmetic of the definition."""
    cfg, grads, rows = parse_hand_case(os.path.join(GOLDEN, "alg4_hand_case_e1.txt"))
    ex = ExactAlg4(cfg["offsets"], cfg["M"], Fraction(cfg["mu"]), Fraction(cfg["eta"]))
    per_step = {}
    for kind, head, cols in rows:
        per_step.setdefault(head[0], []).append((kind, head, cols))
    for t in range(cfg["steps"]):
        res = ex.step([[Fraction(v) for v in grads[(t, i)]] for i in range(cfg["M"])])
        for kind, head, cols in per_step[t]:
            if kind == "worker":
                p, delta, scales = res[head[1]]
                assert [float(v) for v in p] == cols[1]
                assert [float(v) for v in scales] == cols[2]
                assert [1.0 if v < 0 else 0.0 for v in p] == cols[3]
                assert [float(v) for v in ex.e[head[1]]] == cols[5]
                assert [float(v) for v in ex.m[head[1]]] == cols[0]
            else:
                p, delta, scales = res[-1]
                assert [float(v) for v in p] == cols[0]
                assert [float(v) for v in scales] == cols[1]
                assert [float(v) for v in ex.et] == cols[4]
                assert [float(v) for v in ex.x] == cols[5]


# ---------------------------------------------------------------- P2: packing conventions
def test_packing_case_e2():
    vals = {}
    for line in open(os.path.join(GOLDEN, "packing_case_e2.txt")):
        if line.strip() and not line.startswith("#"):
            k, rest = line.split(None, 1)
            vals[k] = rest.split()
    d = int(vals["d"][0])
    g = np.array([(-1) ** k * (k + 1) for k in range(d)], dtype=np.float32)
    o = Oracle([0, d], 1, 0.0, 0.25)
    o.worker_step(0, g)
    assert o.W == 2
    assert o.scales(0).tolist() == [float(vals["scale"][0])]
    assert o.words(0).tolist() == [int(w, 16) for w in vals["words"]]
    expect_e = np.where(np.arange(d) % 2 == 0, g - 20.5, g + 20.5)
    assert np.array_equal(o.residual(0), expect_e.astype(np.float32))
    o.server_step()
    assert o.scales(-1).tolist() == [float(vals["server_scale"][0])]
    assert o.words(-1).tolist() == [int(w, 16) for w in vals["server_words"]]
    assert not o.residual(-1).any()
    # x = -eta * Deltatilde
    assert np.array_equal(o.x, np.where(np.arange(d) % 2 == 0, -0.25 * 20.5, 0.25 * 20.5)
                          .astype(np.float32))


def test_zero_is_positive():
    """Appendix A: signs are mapped to {-1, +1}; zero (and -0) decode to +1."""
    o = Oracle([0, 2], 1, 0.0, 1.0)
    o.worker_step(0, np.array([0.0, 2.0], dtype=np.float32))
    assert o.scales(0).tolist() == [1.0] and o.words(0).tolist() == [0]
    assert o.residual(0).tolist() == [-1.0, 1.0]
    o2 = Oracle([0, 2], 1, 0.0, 1.0)
    o2.worker_step(0, np.array([-0.0, -2.0], dtype=np.float32))
    assert o2.words(0).tolist() == [2]
    o3 = Oracle([0, 3], 1, 0.0, 1.0)          # all-zero block: scale 0, Delta 0, residual 0
    o3.worker_step(0, np.zeros(3, dtype=np.float32))
    assert o3.scales(0).tolist() == [0.0] and o3.words(0).tolist() == [0]
    assert not o3.residual(0).any()


# ---------------------------------------------------------------- P3/P4: Def. 1, Prop. 1
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_compressor_identities(seed):
    """Prop. 1 and its proof: ||C_B(v)-v||^2 = sum_b (||v_b||_2^2 - ||v_b||_1^2/d_b)
    <= (1 - phi(v)) ||v||^2 with phi(v) = min_b ||v_b||_1^2/(d_b ||v_b||_2^2) >= min_b 1/d_b;
    ||Delta_b||_1 = ||v_b||_1; residual = v - Delta (Alg. 4)."""
    rng = np.random.default_rng(seed)
    sizes = [1, 7, 32, 33, 64, 100, 257, 1000]
    off = np.concatenate([[0], np.cumsum(sizes)])
    v = (rng.standard_normal(off[-1]) * np.repeat(rng.uniform(1e-3, 10, len(sizes)), sizes)
         ).astype(np.float32)
    o = Oracle(off, 1, 0.0, 1.0)
    o.worker_step(0, v)                       # mu = 0, e_0 = 0  =>  p = g
    assert np.array_equal(o.last_p, v)
    delta = decode(o.words(0), o.scales(0), off)
    v64 = v.astype(np.longdouble)
    err2 = 0.0
    phi = math.inf
    for b, db in enumerate(sizes):
        blk = v64[off[b]:off[b + 1]]
        l1, l2sq = np.abs(blk).sum(), (blk * blk).sum()
        # L1 preservation
        assert abs(np.abs(delta[off[b]:off[b + 1]]).sum() - l1) <= 1e-6 * l1
        # closed form of the residual norm from the proof of Prop. 1
        e_b = o.residual(0)[off[b]:off[b + 1]].astype(np.longdouble)
        assert abs((e_b * e_b).sum() - (l2sq - l1 * l1 / db)) <= 1e-5 * l2sq
        err2 += (e_b * e_b).sum()
        phi = min(phi, float(l1 * l1 / (db * l2sq)))
    assert phi >= min(1.0 / s for s in sizes) - 1e-12
    assert err2 <= (1 - phi) * float((v64 * v64).sum()) * (1 + 1e-5)
    # e' + Delta = p to one rounding of the subtraction
    s_elem = np.repeat(o.scales(0).astype(np.float64), sizes)
    tol = np.spacing(np.maximum(np.abs(v), s_elem).astype(np.float32))
    assert np.all(np.abs(o.residual(0).astype(np.float64) + delta - v.astype(np.float64)) <= tol)


def test_residual_identity_over_steps():
    """e_{t+1,i} = p_{t,i} - Delta_{t,i} and etilde_{t+1} = ptilde_t - Deltatilde_t (Alg. 4)
    on every call of a multi-step run, decoded independently from the packed output."""
    rng = np.random.default_rng(7)
    sizes = [40, 64, 5, 300]
    off = np.concatenate([[0], np.cumsum(sizes)])
    o = Oracle(off, 3, 0.9, 0.1)
    for t in range(6):
        for i in range(3):
            o.worker_step(i, rng.standard_normal(off[-1]).astype(np.float32))
            p = o.last_p.astype(np.float64)
            delta = decode(o.words(i), o.scales(i), off)
            assert np.allclose(o.residual(i), p - delta, rtol=0, atol=1e-6 * np.abs(p).max())
            assert np.array_equal(delta < 0, p < 0)
        x_before = o.x.copy()
        o.server_step()
        p = o.last_p.astype(np.float64)
        delta = decode(o.words(-1), o.scales(-1), off)
        assert np.allclose(o.residual(-1), p - delta, rtol=0, atol=1e-6 * np.abs(p).max())
        assert np.allclose(o.x, x_before - 0.1 * delta, rtol=0, atol=1e-6)


# ---------------------------------------------------------------- P5: constant magnitude per block
def test_constant_magnitude_blocks_are_compressed_exactly():
    """Section 3.2 example: |v_j| = c_b inside block b  =>  phi = 1, C_B(v) = v, residual 0;
    for the non-block compressor (one block) delta = (1+a)(1-a^B)/(B(1-a)(1+a^B))."""
    Bk, dt, alpha = 6, 16, 0.5
    c = np.array([alpha ** (Bk - 1 - b) for b in range(Bk)])     # c_b / c_{b+1} = alpha
    rng = np.random.default_rng(3)
    sg = rng.choice([-1.0, 1.0], size=Bk * dt)
    v = (np.repeat(c, dt) * sg).astype(np.float32)
    off = np.arange(Bk + 1) * dt
    o = Oracle(off, 1, 0.0, 1.0)
    o.worker_step(0, v)
    assert not o.residual(0).any()
    assert np.array_equal(decode(o.words(0), o.scales(0), off), v.astype(np.float64))
    o1 = Oracle([0, Bk * dt], 1, 0.0, 1.0)
    o1.worker_step(0, v)
    e = o1.residual(0).astype(np.float64)
    delta_emp = 1.0 - (e * e).sum() / (v.astype(np.float64) ** 2).sum()
    delta_formula = (1 + alpha) * (1 - alpha ** Bk) / (Bk * (1 - alpha) * (1 + alpha ** Bk))
    assert abs(delta_emp - delta_formula) < 1e-6


# ---------------------------------------------------------------- P6: Lemma 3 telescoping
def nesterov_sgdm_fp64(grads_per_step, mu, eta):
    """Full-precision distributed SGD with Nesterov momentum (Section 3.3, first display):
    m_i = mu m_i + g_i ; x -= eta * mean_i (mu m_i + g_i)."""
    M, d = len(grads_per_step[0]), len(grads_per_step[0][0])
    m = np.zeros((M, d)); x = np.zeros(d)
    for grads in grads_per_step:
        g = np.asarray(grads, dtype=np.float64)
        m = mu * m + g
        x = x - eta * (mu * m + g).mean(axis=0)
    return x


@pytest.mark.parametrize("M,mu", [(1, 0.0), (2, 0.9), (7, 0.9), (8, 0.5)])
def test_lemma3_error_corrected_iterate(M, mu):
    """Lemma 3: x_T - eta (etilde_T + mean_i e_{T,i}) equals the iterate of uncompressed
    Nesterov SGDM on the same gradients.  Checks the whole two-way path end to end."""
    rng = np.random.default_rng(11 + M)
    sizes = [3, 64, 129, 1000, 31, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)])
    d, eta, T = int(off[-1]), 0.1, 10
    mu32 = float(np.float32(mu)); eta32 = float(np.float32(eta))
    grads = [[(rng.standard_normal(d) * 0.3).astype(np.float32) for _ in range(M)]
             for _ in range(T)]
    o = Oracle(off, M, mu, eta)
    run_steps(o, grads)
    corrected = o.x.astype(np.float64) - eta32 * (
        o.residual(-1).astype(np.float64)
        + np.mean([o.residual(i).astype(np.float64) for i in range(M)], axis=0))
    ref = nesterov_sgdm_fp64(grads, mu32, eta32)
    assert np.abs(corrected - ref).max() <= 1e-5 * np.abs(ref).max()


# ---------------------------------------------------------------- P7: d_b = 1  => identity compressor
def test_unit_blocks_reduce_to_full_precision_sgdm():
    """Section 3.1: with C the identity mapping dist-EF-SGD is full-precision distributed
    SGD.  C_B is the identity when every block has one element."""
    rng = np.random.default_rng(5)
    d, M, mu, eta, T = 50, 4, 0.9, 0.1, 8
    off = np.arange(d + 1)
    grads = [[rng.standard_normal(d).astype(np.float32) for _ in range(M)] for _ in range(T)]
    o = Oracle(off, M, mu, eta)
    run_steps(o, grads)
    for i in range(M):
        assert not o.residual(i).any()
    ref = nesterov_sgdm_fp64(grads, float(np.float32(mu)), float(np.float32(eta)))
    # the server average of M exact values leaves an O(ulp) server residual, carried forward
    assert np.abs(o.x - ref).max() <= 2e-6 * np.abs(ref).max()
    assert np.abs(o.residual(-1)).max() <= 1e-6 * np.abs(ref).max()


# ---------------------------------------------------------------- P8: M = 1
def test_single_worker_server_repeats_worker_message():
    """With M = 1 the server's input is s_b * sign(p): constant magnitude per block, so by
    the Section 3.2 example its compression is exact: same words, same scales, etilde = 0."""
    rng = np.random.default_rng(9)
    sizes = [10, 32, 458, 500]
    off = np.concatenate([[0], np.cumsum(sizes)])
    o = Oracle(off, 1, 0.9, 0.1)
    for t in range(6):
        o.worker_step(0, rng.standard_normal(off[-1]).astype(np.float32))
        o.server_step()
        assert np.array_equal(o.words(-1), o.words(0))
        assert np.array_equal(o.scales(-1), o.scales(0))
        assert not o.residual(-1).any()


def test_single_worker_no_momentum_is_ef_sgd():
    """Algorithm 1 (EF-SGD) with p = eta g + e' equals this method with M = 1, mu = 0 and
    e' = eta e when eta is constant (Section 3.1: the two cases make no difference then)."""
    rng = np.random.default_rng(21)
    d, eta, T = 96, 0.5, 6                     # eta a power of two: scaling is exact
    off = [0, 32, 96]
    o = Oracle(off, 1, 0.0, eta)
    x = np.zeros(d); e = np.zeros(d)
    for t in range(T):
        g = rng.standard_normal(d).astype(np.float32)
        o.worker_step(0, g); o.server_step()
        p = eta * g.astype(np.float64) + e                        # Alg. 1 line 4
        delta = np.empty(d)
        for b in range(2):
            blk = p[off[b]:off[b + 1]]
            delta[off[b]:off[b + 1]] = np.abs(blk).mean() * np.where(blk < 0, -1, 1)
        x -= delta; e = p - delta                                 # Alg. 1 lines 6-7
        assert np.allclose(o.x, x, rtol=0, atol=2e-6)
        assert np.allclose(eta * o.residual(0).astype(np.float64), e, rtol=0, atol=2e-6)


# ---------------------------------------------------------------- P9: Table 1 message sizes
def test_message_size_matches_table1():
    """Table 1: 2Md + 64MB bits per iteration = per direction and worker d sign bits plus one
    float32 per block, when every block is a multiple of 32 elements."""
    sizes = [64, 32, 1024]
    off = np.concatenate([[0], np.cumsum(sizes)])
    o = Oracle(off, 2, 0.9, 0.1)
    assert 32 * (o.W + o.B) == off[-1] + 32 * o.B
    assert o.words(0).nbytes * 8 + o.scales(0).nbytes * 8 == off[-1] + 32 * len(sizes)
    o2 = Oracle([0, 33, 34], 1, 0.9, 0.1)      # every block starts on a word boundary
    assert o2.W == 3


# ---------------------------------------------------------------- P10: brute force, d <= 64
@pytest.mark.parametrize("seed", range(4))
def test_exact_rationals_on_dyadic_inputs(seed):
    rng = np.random.default_rng(100 + seed)
    sizes = [[4, 8, 4], [16, 16], [2, 2, 4, 8, 16, 32], [1, 1, 2, 4]][seed]
    off = [0] + list(np.cumsum(sizes))
    d, M, T = off[-1], [2, 3, 4, 1][seed], 3
    mu, eta = Fraction(1, 2), Fraction(1, 4)
    o = Oracle(off, M, float(mu), float(eta))
    ex = ExactAlg4(off, M, mu, eta)
    for t in range(T):
        grads = [rng.integers(-16, 17, size=d) / 4.0 for _ in range(M)]
        res = ex.step([[Fraction(float(v)) for v in g] for g in grads])
        for i in range(M):
            o.worker_step(i, grads[i].astype(np.float32))
            p, delta, scales = res[i]
            # block sizes are powers of two, so every quantity stays dyadic and exact
            assert [Fraction(float(v)) for v in o.last_p] == p
            assert [Fraction(float(v)) for v in o.scales(i)] == scales
            assert [Fraction(float(v)) for v in o.residual(i)] == ex.e[i]
            assert [Fraction(v) for v in decode(o.words(i), o.scales(i), off)] == delta
        o.server_step()
        p, delta, scales = res[-1]
        if all(Fraction(float(np.float32(float(v)))) == v for v in p):   # still representable
            assert [Fraction(float(v)) for v in o.last_p] == p
            assert [Fraction(float(v)) for v in o.scales(-1)] == scales
            assert [Fraction(float(v)) for v in o.x] == ex.x
        else:
            assert np.allclose(o.x, [float(v) for v in ex.x], rtol=1e-6, atol=1e-7)


def test_scale_and_sign_minimise_l2_error_by_enumeration():
    """The proof of Prop. 1 expands ||s*sigma - v||^2; over all sigma in {-1,+1}^n and all s
    the minimum is at sigma = sign(v), s = ||v||_1/n.  Enumerate for n <= 10."""
    rng = np.random.default_rng(42)
    for n in (1, 2, 5, 10):
        v = rng.standard_normal(n).astype(np.float32)
        o = Oracle([0, n], 1, 0.0, 1.0)
        o.worker_step(0, v)
        s_or = float(o.scales(0)[0])
        sig_or = np.where(decode(o.words(0), [1.0], [0, n]) < 0, -1.0, 1.0)
        best = (math.inf, None, None)
        for sig in itertools.product((-1.0, 1.0), repeat=n):
            sig = np.array(sig)
            s = max(float(sig @ v) / n, 0.0)            # optimal non-negative s for this sigma
            err = float(((s * sig - v) ** 2).sum())
            if err < best[0]:
                best = (err, s, sig)
        assert np.array_equal(best[2], sig_or)
        assert abs(best[1] - s_or) <= 1e-6 * max(1.0, s_or)


# ---------------------------------------------------------------- P11: statistics
def test_scale_statistics_gaussian_and_laplace():
    """For iid N(0, sigma^2) a block's mean |.| tends to sigma*sqrt(2/pi) and phi to 2/pi; for
    Laplace(b) to b and 1/2.  At t = 0, p = (1 + mu + mu... ) g = (mu(1)+1) g since m_0 = g."""
    rng = np.random.default_rng(1234)
    n, sigma, mu = 1 << 16, 0.37, 0.9
    g = (rng.standard_normal(n) * sigma).astype(np.float32)
    o = Oracle([0, n], 1, mu, 0.1)
    o.worker_step(0, g)
    assert abs(o.scales(0)[0] / ((1 + mu) * sigma * math.sqrt(2 / math.pi)) - 1) < 0.01
    e = o.residual(0).astype(np.float64); p = o.last_p.astype(np.float64)
    assert abs((1 - (e * e).sum() / (p * p).sum()) - 2 / math.pi) < 0.01
    lap = rng.laplace(0.0, 0.02, size=n).astype(np.float32)
    o2 = Oracle([0, n], 1, 0.0, 0.1)
    o2.worker_step(0, lap)
    assert abs(o2.scales(0)[0] / 0.02 - 1) < 0.02
    e = o2.residual(0).astype(np.float64); p = lap.astype(np.float64)
    assert abs((1 - (e * e).sum() / (p * p).sum()) - 0.5) < 0.02


# ---------------------------------------------------------------- mu = 0 is Algorithm 3
def test_zero_momentum_is_blocksgd():
    """Section 4: dist-EF-blockSGD is the mu = 0 case: p = g + e, momentum buffer = g."""
    rng = np.random.default_rng(2)
    off = [0, 48, 100]
    o = Oracle(off, 2, 0.0, 0.1)
    e_prev = [np.zeros(100, dtype=np.float32) for _ in range(2)]
    for t in range(4):
        for i in range(2):
            g = rng.standard_normal(100).astype(np.float32)
            o.worker_step(i, g)
            assert np.array_equal(o.momentum(i), g)
            assert np.array_equal(o.last_p, g + e_prev[i])
            e_prev[i] = o.residual(i).copy()
        o.server_step()


# ---------------------------------------------------------------- hint protocol and misuse
def test_hint_adoption_only_inside_zone():
    n = 64
    g = np.linspace(1.0, 2.0, n).astype(np.float32)
    g[5] = 1e-9          # |p| far below 1e-6 * scale
    g[6] = -1e-9
    o_plain = Oracle([0, n], 1, 0.0, 0.1)
    o_plain.worker_step(0, g)
    own = o_plain.words(0).copy()
    assert (own[0] >> 6) & 1 == 1 and (own[0] >> 5) & 1 == 0
    # identical hint: nothing adopted
    o = Oracle([0, n], 1, 0.0, 0.1)
    assert len(o.worker_step(0, g, hint=own)) == 0
    # flipped in-zone bit (element 5) and flipped out-of-zone bit (element 20)
    hint = own.copy(); hint[0] ^= (1 << 5) | (1 << 20)
    o = Oracle([0, n], 1, 0.0, 0.1)
    adopted = o.worker_step(0, g, hint=hint)
    assert adopted.tolist() == [5]
    assert o.words(0)[0] == own[0] ^ (1 << 5)
    s = o.scales(0)[0]
    assert o.residual(0)[5] == np.float32(g[5]) + s          # took the "negative" branch
    assert o.residual(0)[20] == g[20] - s                    # ignored outside the zone


def test_call_order_is_enforced():
    o = Oracle([0, 4], 2, 0.9, 0.1)
    g = np.ones(4, dtype=np.float32)
    with pytest.raises(RuntimeError):
        o.server_step()
    o.worker_step(1, g)
    with pytest.raises(RuntimeError):
        o.worker_step(1, g)
    with pytest.raises(RuntimeError):
        o.server_step()
    o.worker_step(0, g)
    o.server_step()
    assert o.t == 1
    with pytest.raises(ValueError):
        Oracle([0, 2, 2], 1, 0.9, 0.1)        # empty block
    with pytest.raises(ValueError):
        Oracle([0, 4], 1, 1.0, 0.1)           # mu must be < 1


# ---------------------------------------------------------------- property test, exact rationals
from hypothesis import given, settings, strategies as st


@settings(max_examples=40, deadline=None, derandomize=True)
@given(st.lists(st.sampled_from([1, 2, 4, 8, 16, 32, 64]), min_size=1, max_size=5),
       st.sampled_from([1, 2, 4]), st.sampled_from([0.0, 0.25, 0.5]), st.integers(0, 2 ** 31 - 1))
def test_property_two_exact_steps_on_random_dyadic_problems(sizes, M, mu, seed):
    """Random layouts with power-of-two blocks and worker counts (so scales and the server
    average stay dyadic) and dyadic gradients: every quantity of two full steps must equal exact
    rational arithmetic.  (With other M the division by M is inexact, exact cancellations in
    ptilde turn into +-tiny values and the sign there is legitimately not unique.)"""
    rng = np.random.default_rng(seed)
    off = [0] + list(np.cumsum(sizes))
    d = off[-1]
    o = Oracle(off, M, mu, 0.5)
    ex = ExactAlg4(off, M, Fraction(mu), Fraction(1, 2))
    for t in range(2):
        grads = [rng.integers(-8, 9, size=d) / 2.0 for _ in range(M)]
        res = ex.step([[Fraction(float(v)) for v in g] for g in grads])
        for i in range(M):
            o.worker_step(i, grads[i].astype(np.float32))
            p, delta, scales = res[i]
            assert [Fraction(float(v)) for v in o.last_p] == p
            assert [Fraction(float(v)) for v in o.scales(i)] == scales
            assert [Fraction(v) for v in decode(o.words(i), o.scales(i), off)] == delta
            assert [Fraction(float(v)) for v in o.residual(i)] == ex.e[i]
        o.server_step()
        p, delta, scales = res[-1]
        assert [Fraction(float(v)) for v in o.last_p] == p
        assert [Fraction(float(v)) for v in o.scales(-1)] == scales
        assert [Fraction(float(v)) for v in o.residual(-1)] == ex.et
        assert [Fraction(float(v)) for v in o.x] == ex.x
