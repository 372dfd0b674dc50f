"""Exhaustive pins for the truncation-free scale rule (Section 3.1) and for the two rounding modes
(appendix "Rounding and Gradient Propagation")."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from tests.exact import (E2M1_MAGNITUDES, Q_P, bf16_fraction, nearest_even_code, pow2,
                         scale_exponent_exact)

ALL_POSITIVE_FINITE_BF16 = [b for b in range(1, 0x7F80)]


def _bf16_float(bits):
    return float(bf16_fraction(bits))


def test_scale_rule_exhaustive_against_exact_rational_arithmetic():
    # S = 2^ceil(log2(2M/(Qp-Qn))) for every positive finite BF16 maximum M (32 639 values).
    for bits in ALL_POSITIVE_FINITE_BF16:
        M = bf16_fraction(bits)
        assert oracle.scale_exponent(float(M)) == scale_exponent_exact(M), hex(bits)


def test_scale_rule_against_floating_log2_away_from_boundaries():
    # The printed formula evaluated with a floating log2; skipped only where log2 lands within
    # rounding distance of an integer (M = 6*2^k), which the exact test above covers.
    for bits in ALL_POSITIVE_FINITE_BF16[::7]:
        M = _bf16_float(bits)
        t = math.log2(2.0 * M / 12.0)
        if abs(t - round(t)) < 1e-9:
            continue
        assert oracle.scale_exponent(M) == max(-127, math.ceil(t))


def test_scale_rule_against_cuda_e8m0_conversion(library_pins):
    # Library pin: UE8M0 encode of M/6 with the exponent rounded up.
    for bits in ALL_POSITIVE_FINITE_BF16[::3]:
        M = _bf16_float(bits)
        ratio = np.float32(M) / np.float32(6.0)
        if float(ratio) * 6.0 != M or ratio < 2.0 ** -126:    # M/6 not exact in fp32 or subnormal: skip
            continue
        assert oracle.scale_exponent(M) + 127 == library_pins.pin_e8m0_encode_ceil(float(ratio)), hex(bits)


def test_scale_special_cases():
    assert oracle.scale_exponent(0.0) == -127                 # all-zero block
    assert oracle.scale_exponent(6.0) == 0                    # M = Qp -> S = 1
    assert oracle.scale_exponent(6.0 + 2.0 ** -5) == 1        # one BF16 ulp above (6 + 1/32)
    assert oracle.scale_exponent(3.0) == -1 and oracle.scale_exponent(3.0 + 2 ** -6) == 0
    assert oracle.scale_exponent(_bf16_float(0x7F7F)) == 126  # largest finite BF16: code 253


def test_truncation_free_no_value_exceeds_qp():
    # Section 3.1: with the truncation-free scale nothing clips: M/S <= Qp for every M, and the
    # scale is the smallest such power of two unless clamped at 2^-127.
    for bits in ALL_POSITIVE_FINITE_BF16:
        M = bf16_fraction(bits)
        e = oracle.scale_exponent(float(M))
        assert M / pow2(e) <= Q_P
        if e > -127:
            assert M / pow2(e - 1) > Q_P


def _values_up_to_qp():
    # every BF16 value v in [0, 6]
    return [0] + [b for b in ALL_POSITIVE_FINITE_BF16 if bf16_fraction(b) <= 6]


def test_round_nearest_exhaustive():
    for bits in _values_up_to_qp():
        v = bf16_fraction(bits)
        assert oracle.round_nearest(float(v)) == nearest_even_code(v), hex(bits)


def test_round_nearest_ties_and_library(library_pins):
    # midpoints go to the even code
    assert [oracle.round_nearest(v) for v in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0)] == [0, 2, 2, 4, 4, 6, 6]
    for bits in _values_up_to_qp():
        v = _bf16_float(bits) if bits else 0.0
        assert oracle.round_nearest(v) == library_pins.pin_fp4_encode_rn(v)


def test_stochastic_rounding_preserves_expectation_exhaustively():
    # E[roundS(x)] = x (Section 3.1), checked by enumerating all 256 random bytes for every BF16
    # v in [0, 6]: the result is always one of the two neighbours, monotone in the byte, and the
    # mean over the 256 equally likely bytes equals v exactly whenever 256*p is an integer
    # (every v >= 0.25); below that the mean lies in (v - step/256, v].
    for bits in _values_up_to_qp():
        v = bf16_fraction(bits)
        lo = max(c for c in range(8) if E2M1_MAGNITUDES[c] <= v)
        codes = [oracle.round_stochastic(float(v), r) for r in range(256)]
        assert set(codes) <= {lo, min(lo + 1, 7)}
        assert codes == sorted(codes)
        mean = sum(E2M1_MAGNITUDES[c] for c in codes) / 256
        if lo == 7:
            assert mean == 6
            continue
        step = E2M1_MAGNITUDES[lo + 1] - E2M1_MAGNITUDES[lo]
        if v >= Fraction(1, 4) or v == 0:
            assert mean == v, hex(bits)
        else:
            assert v - step / 256 < mean <= v, hex(bits)


def test_stochastic_rounding_never_moves_exact_values():
    for c in range(8):
        assert all(oracle.round_stochastic(float(E2M1_MAGNITUDES[c]), r) == c for r in range(256))


def test_mxfp8_scale_rule_exhaustive():
    for bits in ALL_POSITIVE_FINITE_BF16:
        M = bf16_fraction(bits)
        assert oracle.mxfp8_scale_exponent(float(M)) == scale_exponent_exact(M, Fraction(448)), hex(bits)


def test_e4m3_round_nearest_against_torch_and_cuda(library_pins):
    import torch
    # every BF16 value in [0, 448] (step over the dense low range to keep the run short)
    vals = [b for b in ALL_POSITIVE_FINITE_BF16 if bf16_fraction(b) <= 448]
    vals = [0] + vals[::5] + vals[-400:]
    f = torch.tensor([_bf16_float(b) if b else 0.0 for b in vals], dtype=torch.float32)
    ref = f.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for b, r, x in zip(vals, ref, f.tolist()):
        mine = oracle.round_nearest_e4m3(x)
        assert mine == int(r) == library_pins.pin_e4m3_encode_rn(x), hex(b)
