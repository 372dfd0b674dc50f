"""Exact rational re-derivations used to pin the oracle (tests only).

Everything here is written with ``fractions.Fraction`` straight from the paper's formulas, with no
code shared with the C oracle or the CUDA library.
"""
from fractions import Fraction

E2M1_MAGNITUDES = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3),
                   Fraction(4), Fraction(6)]   # Section 2: E2M1, the MXFP4 element format (OCP MX v1.0)
Q_P, Q_N = Fraction(6), Fraction(-6)


def bf16_fraction(bits: int) -> Fraction:
    """Exact value of a finite BF16 bit pattern."""
    s, be, m = (bits >> 15) & 1, (bits >> 7) & 0xFF, bits & 0x7F
    assert be != 0xFF
    mag = Fraction(m, 128) * Fraction(2) ** (-126) if be == 0 else (1 + Fraction(m, 128)) * Fraction(2) ** (be - 127)
    return -mag if s else mag


def pow2(e: int) -> Fraction:
    return Fraction(2) ** e


def scale_exponent_exact(M: Fraction, qmax: Fraction = Q_P) -> int:
    """ceil(log2(2M/(Qp-Qn))) clamped to [-127, 127], by exact comparison (Section 3.1)."""
    ratio = 2 * M / (2 * qmax)
    if ratio <= pow2(-127):
        return -127
    e = -127
    while pow2(e) < ratio:   # smallest e with 2^e >= ratio  ==  ceil(log2 ratio)
        e += 1
    return min(e, 127)


def nearest_even_code(v: Fraction) -> int:
    best, bestd = 0, abs(v - E2M1_MAGNITUDES[0])
    for c in range(1, 8):
        d = abs(v - E2M1_MAGNITUDES[c])
        if d < bestd or (d == bestd and c % 2 == 0 and best % 2 == 1):
            best, bestd = c, d
    return best


def stochastic_code(v: Fraction, r8: int) -> int:
    lo = max(c for c in range(8) if E2M1_MAGNITUDES[c] <= v)
    if lo == 7:
        return 7
    p = (v - E2M1_MAGNITUDES[lo]) / (E2M1_MAGNITUDES[lo + 1] - E2M1_MAGNITUDES[lo])
    return lo + 1 if (256 * p).__floor__() + r8 >= 256 else lo
