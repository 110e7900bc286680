"""Pins for the oracle's per-block diagnostics (the quantities behind Fig. 1 / Section 3.2)."""
import math

import numpy as np
import pytest

from oracle import Oracle
from paper_1905_10936_b200 import workloads as wl


def phi_delta_cv(diag, sizes):
    """phi(p) (Prop. 1), delta of the non-block compressor (Section 3.2), CV of |g| per block."""
    sizes = np.asarray(sizes, dtype=np.float64)
    p1, p2, g1, g2 = diag.T
    phi_b = p1 * p1 / (sizes * p2)
    delta = p1.sum() ** 2 / (sizes.sum() * p2.sum())
    cv = np.sqrt(np.maximum(sizes * g2 / (g1 * g1) - 1.0, 0.0))
    return phi_b, delta, cv


def test_sums_match_numpy_and_the_residual_norm_of_prop1():
    """||e'_b||_2^2 = ||p_b||_2^2 - ||p_b||_1^2 / d_b (proof of Prop. 1) ties the recorded sums to
    the residual the oracle keeps, which is computed without them."""
    rng = np.random.default_rng(0)
    sizes = [5, 64, 333, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)])
    o = Oracle(off, 2, 0.9, 0.1, diagnostics=True)
    for t in range(3):
        for i in range(2):
            g = (rng.standard_normal(off[-1]) * 0.7).astype(np.float32)
            o.worker_step(i, g)
            dg = o.diagnostics(i)
            p = o.last_p.astype(np.float64); e = o.residual(i).astype(np.float64)
            for b, db in enumerate(sizes):
                sl = slice(off[b], off[b + 1])
                assert math.isclose(dg[b, 0], np.abs(p[sl]).sum(), rel_tol=1e-13)
                assert math.isclose(dg[b, 1], (p[sl] ** 2).sum(), rel_tol=1e-13)
                assert math.isclose(dg[b, 2], np.abs(g[sl].astype(np.float64)).sum(), rel_tol=1e-13)
                assert math.isclose(dg[b, 3], (g[sl].astype(np.float64) ** 2).sum(), rel_tol=1e-13)
                assert math.isclose((e[sl] ** 2).sum(), dg[b, 1] - dg[b, 0] ** 2 / db, rel_tol=1e-5)
                assert math.isclose(float(o.scales(i)[b]), dg[b, 0] / db, rel_tol=1e-6)
        o.server_step()


def test_toy_example_of_section_3_2():
    """Equal blocks, constant magnitude per block, ratio alpha between consecutive blocks:
    phi = 1 and delta = (1+a)(1-a^B) / (B (1-a)(1+a^B)); CV of |g| is 0."""
    Bk, dt, alpha = 8, 32, 0.5
    c = np.array([alpha ** (Bk - 1 - b) for b in range(Bk)])
    rng = np.random.default_rng(4)
    v = (np.repeat(c, dt) * rng.choice([-1.0, 1.0], size=Bk * dt)).astype(np.float32)
    o = Oracle(np.arange(Bk + 1) * dt, 1, 0.0, 0.1, diagnostics=True)
    o.worker_step(0, v)                        # mu = 0, e = 0  =>  p = g = v
    phi_b, delta, cv = phi_delta_cv(o.diagnostics(0), [dt] * Bk)
    assert np.allclose(phi_b, 1.0, rtol=0, atol=1e-12)
    assert abs(delta - (1 + alpha) * (1 - alpha ** Bk) / (Bk * (1 - alpha) * (1 + alpha ** Bk))) < 1e-12
    assert np.all(cv < 1e-6)


def test_gaussian_and_laplace_limits():
    """iid N(0, s^2): phi -> 2/pi, CV(|g|) -> sqrt(pi/2 - 1); Laplace: phi -> 1/2, CV -> 1."""
    n = 1 << 17
    rng = np.random.default_rng(9)
    o = Oracle([0, n, 2 * n], 1, 0.0, 0.1, diagnostics=True)
    g = np.concatenate([rng.standard_normal(n) * 0.3, rng.laplace(0, 0.02, n)]).astype(np.float32)
    o.worker_step(0, g)
    phi_b, delta, cv = phi_delta_cv(o.diagnostics(0), [n, n])
    assert abs(phi_b[0] - 2 / math.pi) < 0.01 and abs(cv[0] - math.sqrt(math.pi / 2 - 1)) < 0.01
    assert abs(phi_b[1] - 0.5) < 0.01 and abs(cv[1] - 1.0) < 0.02
    assert delta < min(phi_b)                 # mixing blocks of different magnitude lowers delta


def test_blockwise_phi_beats_nonblock_delta_on_the_resnet20_layout():
    """Section 3.2, point (ii): with per-tensor magnitudes phi(v) >> ||v||_1^2/(d ||v||_2^2)."""
    w = wl.make_workload(2)
    o = Oracle(w.offsets, 1, 0.9, 0.1, diagnostics=True)
    o.worker_step(0, w.draw_grad(0, 0, "cpu").numpy())
    phi_b, delta, cv = phi_delta_cv(o.diagnostics(0), w.sizes)
    assert phi_b.min() > 0.45 and delta < 0.6 * phi_b.min()
    assert phi_b.min() >= 1.0 / max(w.sizes)


def test_diagnostics_are_off_by_default_and_change_no_result():
    """The sums are not part of Algorithm 4: an oracle that records them and one that does not
    produce identical messages and state, and the latter leaves the diagnostic rows at zero."""
    rng = np.random.default_rng(21)
    sizes = [7, 64, 1000]
    off = np.concatenate([[0], np.cumsum(sizes)])
    a, b = Oracle(off, 2, 0.9, 0.1), Oracle(off, 2, 0.9, 0.1, diagnostics=True)
    for t in range(3):
        for i in range(2):
            g = rng.standard_normal(off[-1]).astype(np.float32)
            a.worker_step(i, g); b.worker_step(i, g)
            assert np.array_equal(a.words(i), b.words(i)) and np.array_equal(a.scales(i), b.scales(i))
            assert not a.diagnostics(i).any() and b.diagnostics(i).all()
        a.server_step(); b.server_step()
    assert np.array_equal(a.x, b.x) and np.array_equal(a.residual(-1), b.residual(-1))
