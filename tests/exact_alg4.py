"""Exact-rational evaluation of Algorithm 4 with the blockwise compressor (Section 3.2).

Brute-force pin for the oracle: Python ``fractions`` carry no rounding at all, so on dyadic
inputs (where binary32 is exact too) the two must agree exactly.  Written directly from the
mathematical statement: vectors are lists of Fractions, the compressor is the definition
C_B(v)_j = (||v_b||_1 / d_b) * sign(v_j).
"""
from fractions import Fraction


def sgn(v):
    return -1 if v < 0 else 1          # Appendix A: signs live in {-1, +1}


def compress(v, offsets):
    """Returns (Delta, scales) of the blockwise compressor."""
    delta, scales = [], []
    for b in range(len(offsets) - 1):
        blk = v[offsets[b]:offsets[b + 1]]
        s = sum(abs(t) for t in blk) / len(blk)
        scales.append(s)
        delta += [s * sgn(t) for t in blk]
    return delta, scales


class ExactAlg4:
    def __init__(self, offsets, M, mu, eta):
        self.off = list(offsets)
        self.d = self.off[-1]
        self.M, self.mu, self.eta = M, Fraction(mu), Fraction(eta)
        zero = [Fraction(0)] * self.d
        self.x = list(zero)
        self.m = [list(zero) for _ in range(M)]
        self.e = [list(zero) for _ in range(M)]
        self.et = list(zero)

    def step(self, grads):
        """grads: M lists of Fractions.  Returns per-worker and server (p, Delta, scales)."""
        out = []
        deltas = []
        for i in range(self.M):
            g = [Fraction(t) for t in grads[i]]
            self.m[i] = [self.mu * a + b for a, b in zip(self.m[i], g)]
            p = [self.mu * a + b + c for a, b, c in zip(self.m[i], g, self.e[i])]
            delta, scales = compress(p, self.off)
            self.e[i] = [a - b for a, b in zip(p, delta)]
            deltas.append(delta)
            out.append((p, delta, scales))
        pt = [sum(dl[j] for dl in deltas) / self.M + self.et[j] for j in range(self.d)]
        dt, st = compress(pt, self.off)
        self.et = [a - b for a, b in zip(pt, dt)]
        self.x = [a - self.eta * b for a, b in zip(self.x, dt)]
        out.append((pt, dt, st))
        return out
