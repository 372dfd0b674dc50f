"""Pins for the GEMM oracle (Section 3, "Application to linear layers") and the MXFP8 operand oracle
(Section 3.2)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2607_24953_b200 import workloads
from tests.exact import bf16_fraction, pow2, scale_exponent_exact


def _rand_bits(seed, rows, cols, spread=1.0):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((rows, cols)) * np.exp(rng.standard_normal((rows, 1)) * spread)).astype(np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16)


def _deq(bits, mode=oracle.MODE_NEAREST, seed=0, tid=0):
    q_rm, _, s = oracle.quantize2d(bits, mode, seed, tid, want_t=False)
    return oracle.dequantize2d(q_rm, s, *bits.shape)


def test_products_against_pure_python_sums():
    # tiny case, every output element summed with exact rationals
    x, w, dy = _deq(_rand_bits(1, 5, 40)), _deq(_rand_bits(2, 7, 40)), _deq(_rand_bits(3, 5, 7))
    F = lambda m: [[Fraction(v) for v in r] for r in m]
    fx, fw, fdy = F(x), F(w), F(dy)
    y = oracle.gemm_fwd(x, w)
    dx = oracle.gemm_dgrad(dy, w)
    dw = oracle.gemm_wgrad(dy, x)
    for t in range(5):
        for n in range(7):
            assert y[t, n] == pytest.approx(float(sum(fx[t][k] * fw[n][k] for k in range(40))), rel=1e-14, abs=1e-300)
        for k in range(40):
            assert dx[t, k] == pytest.approx(float(sum(fdy[t][n] * fw[n][k] for n in range(7))), rel=1e-14, abs=1e-300)
    for n in range(7):
        for k in range(40):
            assert dw[n, k] == pytest.approx(float(sum(fdy[t][n] * fx[t][k] for t in range(5))), rel=1e-14, abs=1e-300)


def test_library_matmul_agrees_with_definition_loop():
    x, w, dy = _deq(_rand_bits(4, 48, 96)), _deq(_rand_bits(5, 64, 96)), _deq(_rand_bits(6, 48, 64))
    assert np.allclose(oracle.gemm_fwd(x, w), oracle.gemm_nt_definition(x, w), rtol=1e-13, atol=0)
    assert np.allclose(oracle.gemm_dgrad(dy, w), oracle.gemm_nt_definition(dy, np.ascontiguousarray(w.T)), rtol=1e-12, atol=1e-300)
    assert np.allclose(oracle.gemm_wgrad(dy, x), oracle.gemm_nt_definition(np.ascontiguousarray(dy.T), np.ascontiguousarray(x.T)), rtol=1e-12, atol=1e-300)


def test_gradient_identities():
    # <dY, X W^T> = <dY W, X> = <dY^T X, W>: the three products are the forward map and its two adjoints.
    x, w, dy = _deq(_rand_bits(7, 33, 64)), _deq(_rand_bits(8, 40, 64)), _deq(_rand_bits(9, 33, 40))
    a = (dy * oracle.gemm_fwd(x, w)).sum()
    b = (oracle.gemm_dgrad(dy, w) * x).sum()
    c = (oracle.gemm_wgrad(dy, x) * w).sum()
    assert a == pytest.approx(b, rel=1e-12) and a == pytest.approx(c, rel=1e-12)


def test_exact_integer_special_case():
    # operands on the E2M1 grid times one power of two: every partial sum is a small integer multiple of
    # 0.25 * 2^(ea+eb), so the result is exact in any accumulation order and precision >= fp32.
    rng = np.random.default_rng(10)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    a = rng.choice(grid, size=(16, 64)) * rng.choice([-1, 1], size=(16, 64)) * 2.0 ** -3
    b = rng.choice(grid, size=(24, 64)) * rng.choice([-1, 1], size=(24, 64)) * 2.0 ** 5
    bits = lambda m: (m.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    ad, bd = _deq(bits(a)), _deq(bits(b))
    assert np.array_equal(ad, a) and np.array_equal(bd, b)        # grid values survive quantization
    y = oracle.gemm_fwd(ad, bd)
    assert np.array_equal(y, (a.astype(np.float32) @ b.astype(np.float32).T).astype(np.float64))
    assert np.array_equal(y * 4 * 2.0 ** -2, np.round(y * 4 * 2.0 ** -2))


def test_grouped_products_match_per_group_dense_products():
    counts = np.array([3, 0, 5, 2])
    offs = workloads.padded_row_offsets(counts, pad=4)
    assert list(offs) == [0, 4, 4, 12, 16]
    T = int(offs[-1])
    x = _deq(_rand_bits(11, T, 32))
    w = _deq(_rand_bits(12, 4 * 8, 32))
    y = oracle.grouped(oracle.gemm_fwd, x, w, offs)
    assert y.shape == (T, 8)
    assert np.array_equal(y[4:12], oracle.gemm_fwd(x[4:12], w[16:24]))
    dy = _deq(_rand_bits(13, T, 8))
    dw = oracle.grouped_wgrad(dy, x, offs)
    assert dw.shape == (32, 32) and not dw[8:16].any()              # empty group: zero gradient
    assert np.array_equal(dw[24:32], oracle.gemm_wgrad(dy[12:16], x[12:16]))


def test_bf16_round():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -8 + 2 ** -20, 1.0 + 3 * 2 ** -8, -3.14159, 0.0])
    import torch
    ref = torch.tensor(v, dtype=torch.float32).to(torch.bfloat16).double().numpy()
    assert np.array_equal(oracle.bf16_round(v), ref)


# ------------------------------------------------------------------------------------------ MXFP8

def test_mxfp8_against_exact_brute_force_and_torch():
    import torch
    bits = _rand_bits(20, 9, 70, spread=2.0)
    bits[0, :32] = 0
    bits[1, 3] = 0x43E0            # 448 exactly
    bits[2, 3] = 0x43E1            # one ulp above 448
    q, s = oracle.mxfp8_quantize1d(bits)
    assert q.shape == (9, 70) and s.shape == (9, 3)
    for i in range(9):
        for b in range(3):
            cols = range(32 * b, min(32 * b + 32, 70))
            M = max(abs(bf16_fraction(int(bits[i, j]))) for j in cols)
            e = scale_exponent_exact(M, Fraction(448))
            assert s[i, b] == e + 127
            scaled = torch.tensor([float(bf16_fraction(int(bits[i, j])) / pow2(e)) for j in cols], dtype=torch.float32)
            assert (scaled.abs() <= 448).all()                     # truncation-free: never saturates
            ref = scaled.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            got = q[i, 32 * b:32 * b + len(ref)]
            assert np.array_equal(got & 0x7F, ref & 0x7F)
            nz = (got & 0x7F) != 0
            assert np.array_equal(got[nz] >> 7, ref[nz] >> 7)
    deq = oracle.mxfp8_dequantize(q, s)
    src = np.array([[float(bf16_fraction(int(b))) for b in r] for r in bits])
    assert (np.abs(deq - src) <= np.abs(src) * 2.0 ** -4 + 2.0 ** -130).all()   # 3 mantissa bits: rel err <= 2^-4
    assert s[0, 0] == 0 and not q[0, :32].any()


def test_mxfp8_products_use_per_row_block_scales():
    x = oracle.mxfp8_dequantize(*oracle.mxfp8_quantize1d(_rand_bits(21, 6, 64)))
    w = oracle.mxfp8_dequantize(*oracle.mxfp8_quantize1d(_rand_bits(22, 10, 64)))
    assert np.allclose(oracle.gemm_fwd(x, w), oracle.gemm_nt_definition(x, w), rtol=1e-13, atol=0)


def test_mxfp8_transposed_operand_is_the_operand_of_the_transpose():
    """Blocks along the other axis: the transposing form must be the plain form applied to x^T, and decoding it
    must give x^T back within the E4M3 rounding error (relative 2^-4 of the block maximum)."""
    import numpy as np
    from paper_2607_24953_b200 import workloads
    import oracle
    x = workloads.activations_student_t(70, 45, 5, "cpu")
    bits = workloads.bf16_bits(x)
    q, s = oracle.mxfp8_quantize1d_t(bits)
    assert q.shape == (45, 70) and s.shape == (45, 3)
    q2, s2 = oracle.mxfp8_quantize1d(np.ascontiguousarray(bits.T))
    assert np.array_equal(q, q2) and np.array_equal(s, s2)
    back = oracle.mxfp8_dequantize(q, s)
    ref = x.double().numpy().T
    for j in range(45):
        for b in range(3):
            seg = slice(32 * b, min(32 * b + 32, 70))
            m = np.abs(ref[j, seg]).max()
            assert np.abs(back[j, seg] - ref[j, seg]).max() <= m * 2.0 ** -4 + 1e-300
