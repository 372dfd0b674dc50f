"""Pins of the 1D-block (1 x 32) FP4 oracle - the activation layout the paper keeps (Section 3.1) - against things
other than itself: a 1 x 32 block is a 32 x 32 block with a single populated row, so each row must quantize exactly
like the one-row matrix does in the pinned 2D oracle; the scale rule and no-clipping invariants; exact expectation of
the stochastic rounding; and the Figure 1 diagnostic's qualitative claims on synthetic tensors."""
import numpy as np
import pytest

import oracle
from paper_2607_24953_b200 import workloads


def bits_of(t):
    return workloads.bf16_bits(t)


@pytest.mark.parametrize("rows,cols", [(5, 96), (3, 70), (1, 1), (8, 33)])
def test_rows_quantize_like_one_row_matrices_in_the_2d_oracle(rows, cols):
    x = bits_of(workloads.activations_student_t(rows, cols, 41, "cpu"))
    q, s = oracle.quantize1d(x, oracle.MODE_NEAREST)
    for i in range(rows):
        q2, _, s2 = oracle.quantize2d(x[i:i + 1], oracle.MODE_NEAREST, want_t=False)
        assert np.array_equal(q[i:i + 1], q2)
        assert np.array_equal(s[i:i + 1], s2)
    # stochastic: row 0 has the same element indices in both, so the same random bytes
    q, s = oracle.quantize1d(x, oracle.MODE_STOCHASTIC, seed=5, tensor_id=2)
    q2, _, s2 = oracle.quantize2d(x[0:1], oracle.MODE_STOCHASTIC, seed=5, tensor_id=2, want_t=False)
    assert np.array_equal(q[0:1], q2) and np.array_equal(s[0:1], s2)


def test_scale_is_truncation_free_and_tight_per_row_block():
    x = bits_of(workloads.activations_student_t(16, 256, 42, "cpu"))
    vals = oracle.bits_to_double(x)
    q, s = oracle.quantize1d(x)
    deq = oracle.dequantize1d(q, s, 16, 256)
    for i in range(16):
        for b in range(8):
            m = np.abs(vals[i, 32 * b:32 * b + 32]).max()
            S = 2.0 ** (int(s[i, b]) - 127)
            assert m <= 6 * S and (m > 3 * S or m == 0)          # smallest power of two with 6 S >= M
            assert np.abs(deq[i, 32 * b:32 * b + 32]).max() <= 6 * S


def test_stochastic_rounding_mean_over_seeds_approaches_the_input():
    x = bits_of(workloads.activations_student_t(2, 64, 43, "cpu"))
    vals = oracle.bits_to_double(x)
    acc = np.zeros_like(vals)
    n = 400
    for seed in range(n):
        q, s = oracle.quantize1d(x, oracle.MODE_STOCHASTIC, seed=seed, tensor_id=0)
        acc += oracle.dequantize1d(q, s, 2, 64)
    S = np.repeat(2.0 ** (s.astype(np.float64) - 127), 32, axis=1)
    # one step of the local grid is at most 2 S; the mean of n draws is within 4.5 sigma of the input
    assert (np.abs(acc / n - vals) <= 4.5 * S / np.sqrt(n) + S * 2.0 ** -9).all()


def test_transposed_form_keeps_the_rounding_stream_of_the_element():
    x = bits_of(workloads.activations_student_t(40, 70, 44, "cpu"))
    q, s = oracle.quantize1d_t(x, oracle.MODE_STOCHASTIC, seed=9, tensor_id=1)
    assert q.shape == (70, 20) and s.shape == (70, 2)
    # element (i, j) of x sits at (j, i) of the transposed encoding and draws the byte of index i*cols + j
    vals = oracle.bits_to_double(x)
    for (i, j) in ((0, 0), (7, 3), (39, 69), (33, 1)):
        S = 2.0 ** (int(s[j, i // 32]) - 127)
        r8 = oracle.random_byte(9, 1, i * 70 + j)
        mag = oracle.round_stochastic(abs(vals[i, j]) / S, r8)
        code = (q[j, i // 2] >> (4 * (i & 1))) & 0xF
        assert code == ((8 if vals[i, j] < 0 or (x[i, j] >> 15) else 0) | mag)


def test_figure_1_diagnostic_1d_mismatches_2d_does_not():
    # activations with outlier channels: the scale an element gets depends on the axis its 1D block runs along
    x = bits_of(workloads.activations_gauss_outliers(128, 256, 45, "cpu"))
    d = oracle.transposition_diagnostic(x)
    assert not d["scale_exponent_difference_2d"].any()
    assert d["deviation_2d"] == 0.0
    assert np.abs(d["scale_exponent_difference_1d"]).mean() > 0.5
    assert d["deviation_1d"] > 1e-2
