"""Pins for the oracle's rounding conventions where the paper is silent.

The paper fixes none of these (they are readings of this repository, each marked in the
oracle's header), so they cannot be pinned to the paper; they are pinned to hand-built cases in
which the alternatives give a different binary32 result, so that a change of convention on
either side cannot pass unnoticed:
  * the block's L1 sum is accumulated in (at least) binary64 and rounded once,
  * the server adds the workers' scaled signs in ascending worker order,
  * the rescaled residual enters through ONE rounding, p = fl(r*e + u).
Expectations are computed with exact rational arithmetic and a correct rounding to binary32
written out below."""
from fractions import Fraction

import numpy as np

from oracle import Oracle


def round_to_f32(q: Fraction) -> np.float32:
    """Round-to-nearest-even of an exact rational to binary32 (normal range only)."""
    if q == 0:
        return np.float32(0.0)
    sign = -1 if q < 0 else 1
    q = abs(q)
    e = 0
    while q >= 2:
        q /= 2; e += 1
    while q < 1:
        q *= 2; e -= 1
    scaled = q * (1 << 23)                      # in [2^23, 2^24)
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    assert -126 <= e <= 127
    return np.float32(sign * float(n) * 2.0 ** (e - 23))


def test_round_to_f32_helper():
    for v in (1.0, 1.5, 0.1, 3.0e-5, 16777217.0, 1 + 2 ** -24, 1 + 3 * 2 ** -25):
        assert round_to_f32(Fraction(v)) == np.float32(v)
    assert round_to_f32(Fraction(1) + Fraction(1, 2 ** 24)) == np.float32(1.0)            # tie -> even
    assert round_to_f32(Fraction(1) + Fraction(3, 2 ** 24)) == np.float32(1 + 2 ** -22)   # tie -> even


def test_block_sum_is_accumulated_beyond_binary32():
    """|p| = [2^24, 1, 1, 1]: a binary32 running sum stays at 2^24 (each +1 is a tie that rounds
    back), the true sum is 2^24 + 3.  The scale must be the correctly rounded true mean."""
    g = np.array([2.0 ** 24, -1.0, 1.0, -1.0], dtype=np.float32)
    o = Oracle([0, 4], 1, 0.0, 0.1)
    o.worker_step(0, g)                                          # mu = 0, e = 0: p = g
    want = round_to_f32(Fraction(2 ** 24 + 3, 4))
    assert o.scales(0)[0] == want
    assert want != np.float32(np.float32(2.0 ** 24) / np.float32(4.0))      # what a binary32 sum would give


def test_server_adds_workers_in_ascending_order():
    """Three workers whose scaled scales are c = (2^24, 1, 1), all signs positive:
    ((c0 + c1) + c2) = 2^24 in binary32 (two ties), while ((c2 + c1) + c0) = 2^24 + 2."""
    M = 3
    o = Oracle([0, 2], M, 0.0, 0.5)
    for i, s in enumerate((3 * 2.0 ** 24, 3.0, 3.0)):            # scale_i / M = c_i exactly
        o.worker_step(i, np.array([s, s], dtype=np.float32))     # constant magnitude: scale = s
        assert o.scales(i)[0] == np.float32(s)
    o.server_step()
    assert np.all(o.last_p == np.float32(2.0 ** 24))             # ptilde = a + etilde(0)
    assert o.scales(-1)[0] == np.float32(2.0 ** 24)
    rev = np.float32(np.float32(np.float32(1.0) + np.float32(1.0)) + np.float32(2.0 ** 24))
    assert rev == np.float32(2.0 ** 24 + 2)                      # the other order is different


def test_rescaled_residual_enters_with_a_single_rounding():
    """eta changes from 0.3 to 0.07: r = fl(0.3f / 0.07f).  With a residual e and u = mu m + g such
    that fl(fl(r e) + u) differs from fl(r e + u) (about one random case in four), the oracle's
    p must be the latter."""
    eta0, eta1 = np.float32(0.3), np.float32(0.07)
    r = np.float32(eta0 / eta1)
    rng = np.random.default_rng(6)
    checked = 0
    for _ in range(40):
        # step 0: one block of two elements, p = g (mu = 0): residual e = p - scale*sign(p)
        o = Oracle([0, 2], 1, 0.0, float(eta0))
        o.worker_step(0, rng.standard_normal(2).astype(np.float32))
        o.server_step()
        e = o.residual(0).copy()
        o.set_eta(float(eta1))
        u = np.float32(rng.standard_normal())
        one = round_to_f32(Fraction(float(r)) * Fraction(float(e[0])) + Fraction(float(u)))
        two = np.float32(np.float32(r * e[0]) + u)
        o.worker_step(0, np.array([u, 0.0], dtype=np.float32))   # mu = 0: u = g
        assert o.last_p[0] == one
        checked += int(one != two)
    assert checked >= 3, "too few cases separate the two forms"
