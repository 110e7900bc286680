"""Pins for the oracle's stepsize sequence (eta_{t-1}/eta_t residual rescale, Algorithms 2-4)
and weight-decay side path (Appendix A).  Expectations come from hand-worked cases, the
error-corrected-iterate lemma in its general form, and textbook Nesterov SGDM in fp64."""
import os

import numpy as np
import pytest

from oracle import Oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "stepsize_and_decay_hand_cases.txt")


def _rows(case):
    out = []
    for line in open(GOLDEN):
        t = line.split()
        if t and t[0] == case:
            row, key = {}, None
            for tok in t[2:]:
                try:
                    val = float(tok)
                except ValueError:
                    key = tok; row[key] = []
                    continue
                row[key].append(val)
            out.append(row)
    return out


def test_hand_case_stepsize_change():
    rows = _rows("A")
    o = Oracle([0, 2], 1, 0.0, rows[0]["eta"][0])
    for k, r in enumerate(rows):
        if k:
            o.set_eta(r["eta"][0])
        o.worker_step(0, np.array(r["grad"], dtype=np.float32))
        assert o.last_p.tolist() == r["p"]
        assert o.scales(0).tolist() == r["scale"]
        assert o.residual(0).tolist() == r["resid"]
        o.server_step()
        assert o.x.tolist() == r["x"]


def test_hand_case_weight_decay():
    rows = _rows("B")
    o = Oracle([0, 1], 1, 0.5, 0.5)
    o.set_weight_decay(0.5)
    o.x[:] = 4.0
    for r in rows:
        o.worker_step(0, np.zeros(1, dtype=np.float32))
        o.server_step()
        assert o.decay_momentum.tolist() == r["mtilde"]
        assert o.x.tolist() == r["x"]


def _run(o, grads, etas):
    xs = []
    for t, gs in enumerate(grads):
        if t:
            o.set_eta(etas[t])
        xs.append(o.x.astype(np.float64).copy())
        for i, g in enumerate(gs):
            o.worker_step(i, g)
        o.server_step()
    return xs


@pytest.mark.parametrize("schedule", ["step_decay", "warmup", "zigzag"])
def test_error_corrected_iterate_with_changing_stepsize(schedule):
    """General lemma of the appendix: xtilde_t = x_t - eta_{t-1}(etilde_t + mean_i e_{t,i})
    obeys xtilde_{t+1} = xtilde_t - eta_t mean_i(mu m_{t,i} + g_{t,i}); the right-hand side is
    uncompressed Nesterov SGDM with the same stepsize sequence.  Fails if either residual is
    not rescaled by eta_{t-1}/eta_t."""
    rng = np.random.default_rng(5)
    sizes = [7, 64, 300, 1029]
    off = np.concatenate([[0], np.cumsum(sizes)])
    d, M, mu, T = int(off[-1]), 3, 0.9, 9
    etas = {"step_decay": [0.1] * 3 + [0.01] * 3 + [0.001] * 3,
            "warmup": [0.01 * (k + 1) for k in range(T)],
            "zigzag": [0.1, 0.025, 0.2, 0.05, 0.1, 0.4, 0.05, 0.0125, 0.1]}[schedule]
    etas32 = [float(np.float32(e)) for e in etas]
    grads = [[(rng.standard_normal(d) * 0.5).astype(np.float32) for _ in range(M)] for _ in range(T)]
    o = Oracle(off, M, mu, etas[0])
    _run(o, grads, etas)
    corrected = o.x.astype(np.float64) - etas32[-1] * (
        o.residual(-1).astype(np.float64)
        + np.mean([o.residual(i).astype(np.float64) for i in range(M)], axis=0))
    mu32 = float(np.float32(mu))
    m = np.zeros((M, d)); ref = np.zeros(d)
    for t in range(T):
        g = np.asarray(grads[t], dtype=np.float64)
        m = mu32 * m + g
        ref -= etas32[t] * (mu32 * m + g).mean(axis=0)
    assert np.abs(corrected - ref).max() <= 2e-5 * np.abs(ref).max()


def test_constant_stepsize_set_explicitly_changes_nothing():
    rng = np.random.default_rng(1)
    off = [0, 40, 100]
    grads = [[rng.standard_normal(100).astype(np.float32) for _ in range(2)] for _ in range(4)]
    a, b = Oracle(off, 2, 0.9, 0.1), Oracle(off, 2, 0.9, 0.1)
    _run(a, grads, [0.1] * 4)
    for t, gs in enumerate(grads):
        for i, g in enumerate(gs):
            b.worker_step(i, g)
        b.server_step()
    assert np.array_equal(a.x, b.x) and np.array_equal(a.residual(0), b.residual(0))


def test_weight_decay_alone_is_nesterov_on_a_quadratic():
    """Zero gradients: Deltatilde = 0 and the update is Nesterov SGDM on (lambda/2)||x||^2."""
    d, mu, eta, lam, T = 33, 0.9, 0.1, 0.05, 12
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal(d).astype(np.float32)
    o = Oracle([0, 10, d], 2, mu, eta)
    o.set_weight_decay(lam)
    o.x[:] = x0
    z = np.zeros(d, dtype=np.float32)
    _run(o, [[z, z]] * T, [eta] * T)
    mu_, eta_, lam_ = (float(np.float32(v)) for v in (mu, eta, lam))
    x = x0.astype(np.float64); m = np.zeros(d)
    for t in range(T):
        g = lam_ * x
        m = mu_ * m + g
        x = x - eta_ * (mu_ * m + g)
    assert np.abs(o.x - x).max() <= 1e-5 * np.abs(x).max()
    assert not o.residual(-1).any()


def test_weight_decay_with_identity_compressor_is_sgdm_on_g_plus_lambda_x():
    """d_b = 1 makes C_B the identity; momentum is additive (Appendix A), so the scheme equals
    full-precision Nesterov SGDM on the gradient g + lambda x."""
    d, M, mu, eta, lam, T = 24, 3, 0.9, 0.05, 0.1, 8
    rng = np.random.default_rng(8)
    grads = [[rng.standard_normal(d).astype(np.float32) for _ in range(M)] for _ in range(T)]
    o = Oracle(np.arange(d + 1), M, mu, eta)
    o.set_weight_decay(lam)
    _run(o, grads, [eta] * T)
    mu_, eta_, lam_ = (float(np.float32(v)) for v in (mu, eta, lam))
    x = np.zeros(d); m = np.zeros((M, d))
    for t in range(T):
        g = np.asarray(grads[t], dtype=np.float64) + lam_ * x
        m = mu_ * m + g
        x = x - eta_ * (mu_ * m + g).mean(axis=0)
    assert np.abs(o.x - x).max() <= 1e-5 * np.abs(x).max()


def test_error_corrected_iterate_with_weight_decay_and_changing_stepsize():
    """xtilde_{t+1} = xtilde_t - eta_t [ mean_i(mu m_i + g_i) + mu mtilde_t + lambda x_t ]: the
    decay terms are applied uncompressed (Appendix A).  x_t on the right is the oracle's own
    iterate; everything else is recomputed in fp64."""
    rng = np.random.default_rng(13)
    sizes = [5, 96, 700]
    off = np.concatenate([[0], np.cumsum(sizes)])
    d, M, mu, lam, T = int(off[-1]), 2, 0.9, 0.02, 8
    etas = [0.1, 0.1, 0.05, 0.05, 0.2, 0.1, 0.025, 0.025]
    grads = [[(rng.standard_normal(d) * 0.3).astype(np.float32) for _ in range(M)] for _ in range(T)]
    o = Oracle(off, M, mu, etas[0])
    o.set_weight_decay(lam)
    xs = _run(o, grads, etas)
    mu_, lam_ = float(np.float32(mu)), float(np.float32(lam))
    e32 = [float(np.float32(e)) for e in etas]
    m = np.zeros((M, d)); mt = np.zeros(d); ref = np.zeros(d)
    for t in range(T):
        g = np.asarray(grads[t], dtype=np.float64)
        m = mu_ * m + g
        mt = mu_ * mt + lam_ * xs[t]
        ref -= e32[t] * ((mu_ * m + g).mean(axis=0) + mu_ * mt + lam_ * xs[t])
    corrected = o.x.astype(np.float64) - e32[-1] * (
        o.residual(-1).astype(np.float64)
        + np.mean([o.residual(i).astype(np.float64) for i in range(M)], axis=0))
    assert np.abs(corrected - ref).max() <= 2e-5 * np.abs(ref).max()
    assert np.abs(o.decay_momentum - mt).max() <= 1e-5 * np.abs(mt).max()


def test_setters_are_refused_in_the_middle_of_an_iteration():
    o = Oracle([0, 4], 2, 0.9, 0.1)
    o.worker_step(0, np.ones(4, dtype=np.float32))
    with pytest.raises(RuntimeError):
        o.set_eta(0.2)
    with pytest.raises(RuntimeError):
        o.set_weight_decay(0.1)
