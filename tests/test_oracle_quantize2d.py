"""Pins for the oracle's 2D-block quantizer as a whole: brute force on tiny inputs in exact rational
arithmetic, transposition invariance, no clipping, boundary blocks, unbiasedness over 10^4 seeds."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2607_24953_b200 import workloads
from tests.exact import (E2M1_MAGNITUDES, bf16_fraction, nearest_even_code, pow2, scale_exponent_exact)


def _random_bits(rng, rows, cols, scale_spread=True):
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    if scale_spread:
        x *= np.exp(rng.standard_normal((rows, 1)) * 2).astype(np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16)


def _nibbles_rm(q, cols):
    out = np.zeros((q.shape[0], cols), dtype=np.uint8)
    out[:, 0::2] = (q & 0xF)[:, :(cols + 1) // 2]
    out[:, 1::2] = (q >> 4)[:, :cols // 2]
    return out


def _brute_force(bits, mode, seed, tid, transposed_index=False):
    """Whole quantizer re-derived with exact rationals and pure-Python loops."""
    rows, cols = bits.shape
    rt, ct = -(-rows // 32), -(-cols // 32)
    codes = np.zeros((rows, cols), dtype=np.uint8)
    scale = np.zeros((rt, ct), dtype=np.uint8)
    for I in range(rt):
        for J in range(ct):
            blk = [(i, j) for i in range(32 * I, min(32 * I + 32, rows)) for j in range(32 * J, min(32 * J + 32, cols))]
            M = max(abs(bf16_fraction(int(bits[i, j]))) for i, j in blk)
            e = scale_exponent_exact(M)
            scale[I, J] = e + 127
            for i, j in blk:
                b = int(bits[i, j])
                v = abs(bf16_fraction(b)) / pow2(e)
                if mode == oracle.MODE_NEAREST:
                    mag = nearest_even_code(v)
                else:
                    idx = j * rows + i if transposed_index else i * cols + j
                    blkno = idx >> 4
                    out = oracle.philox4x32_10([blkno & 0xFFFFFFFF, blkno >> 32, tid, 0],
                                               [seed & 0xFFFFFFFF, seed >> 32])   # pinned separately
                    r8 = (int(out[(idx >> 2) & 3]) >> (8 * (idx & 3))) & 0xFF
                    lo = max(c for c in range(8) if E2M1_MAGNITUDES[c] <= v)
                    if lo == 7:
                        mag = 7
                    else:
                        p = (v - E2M1_MAGNITUDES[lo]) / (E2M1_MAGNITUDES[lo + 1] - E2M1_MAGNITUDES[lo])
                        mag = lo + 1 if int(256 * p) + r8 >= 256 else lo
                codes[i, j] = ((b >> 15) << 3) | mag
    return codes, scale


@pytest.mark.parametrize("shape", [(32, 32), (33, 31), (1, 1), (64, 96)])
@pytest.mark.parametrize("mode", [oracle.MODE_NEAREST, oracle.MODE_STOCHASTIC])
def test_tiny_inputs_against_exact_brute_force(shape, mode):
    rng = np.random.default_rng(shape[0] * 100 + shape[1])
    bits = _random_bits(rng, *shape)
    q_rm, q_t, scale = oracle.quantize2d(bits, mode, seed=0xDEADBEEF12, tensor_id=5)
    codes, scale_ref = _brute_force(bits, mode, 0xDEADBEEF12, 5)
    assert np.array_equal(scale, scale_ref)
    assert np.array_equal(_nibbles_rm(q_rm, shape[1]), codes)
    assert np.array_equal(_nibbles_rm(q_t, shape[0]), codes.T)      # the second layout is the transpose


def test_adversarial_tiles_against_exact_brute_force():
    # subnormal tiles, maxima exactly 6*2^k and one ulp above, +-0, largest finite BF16
    rng = np.random.default_rng(3)
    bits = _random_bits(rng, 64, 64, scale_spread=False)
    bits[0:32, 0:32] = rng.integers(0, 0x80, size=(32, 32)).astype(np.uint16)            # all subnormal
    bits[0, 0] |= 0x8000
    bits[0:32, 32:64] = 0
    bits[3, 40] = 0x8000                                                                 # -0 in a zero tile
    t = bits[32:64, 0:32]
    t[...] = (t & 0x807F) | (0x3F << 7)                                                  # all in [0.5, 1)
    t[5, 5] = 0x40C0                                                                     # 6.0 exactly
    u = bits[32:64, 32:64]
    u[...] = (u & 0x807F) | (0x3F << 7)
    u[7, 9] = 0x40C1                                                                     # 6 + one ulp
    u[8, 9] = 0x7F7F                                                                     # largest finite
    for mode in (oracle.MODE_NEAREST, oracle.MODE_STOCHASTIC):
        q_rm, q_t, scale = oracle.quantize2d(bits, mode, seed=9, tensor_id=1)
        codes, scale_ref = _brute_force(bits, mode, 9, 1)
        assert np.array_equal(scale, scale_ref)
        assert np.array_equal(_nibbles_rm(q_rm, 64), codes)
        assert np.array_equal(_nibbles_rm(q_t, 64), codes.T)
    assert scale[0, 1] == 0 and scale[1, 0] == 127 and scale[1, 1] == 253
    assert _nibbles_rm(q_rm, 64)[3, 40] == 0x8                                           # sign of -0 kept


@pytest.mark.parametrize("shape", [(96, 160), (70, 45)])
def test_transposition_invariance(shape):
    # S(B_ij) = S(B_ij^T): quantize(A)^T == quantize(A^T) bit for bit (Section 3; appendix
    # "2D Block Scaling and Transposition Consistency").
    rng = np.random.default_rng(11)
    a = _random_bits(rng, *shape)
    at = np.ascontiguousarray(a.T)
    q_rm, q_t, s = oracle.quantize2d(a, oracle.MODE_NEAREST)
    p_rm, p_t, st = oracle.quantize2d(at, oracle.MODE_NEAREST)
    assert np.array_equal(st, s.T)
    assert np.array_equal(p_rm, q_t) and np.array_equal(p_t, q_rm)
    # stochastic: same draws when the transposed call keys its stream on the original element index
    q_rm, q_t, s = oracle.quantize2d(a, oracle.MODE_STOCHASTIC, seed=4, tensor_id=2)
    p_rm, p_t, st = oracle.quantize2d(at, oracle.MODE_STOCHASTIC, seed=4, tensor_id=2,
                                      flags=oracle.FLAG_INDEX_TRANSPOSED)
    assert np.array_equal(st, s.T)
    assert np.array_equal(p_rm, q_t) and np.array_equal(p_t, q_rm)


def test_one_dimensional_blocks_would_not_be_invariant():
    # Section 2.1's failure mode, as a sanity check that the invariance test can fail: with the same
    # scale rule applied per 1x32 row segment, the scales of A and A^T disagree for most elements.
    rng = np.random.default_rng(5)
    a = _random_bits(rng, 64, 64)
    def row_scales(m):
        v = np.array([[abs(float(bf16_fraction(int(b)))) for b in r] for r in m])
        return np.array([[oracle.scale_exponent(v[i, 32 * k:32 * k + 32].max()) for k in range(2)] for i in range(64)])
    fwd = np.repeat(row_scales(a), 32, axis=1)
    bwd = np.repeat(row_scales(np.ascontiguousarray(a.T)), 32, axis=1).T
    assert (fwd != bwd).mean() > 0.3


def test_no_clipping_and_error_bound_on_workload_tensors():
    t = workloads.tiny_layer()
    for name, tensor in t.items():
        bits = workloads.bf16_bits(tensor)
        for mode in (oracle.MODE_NEAREST, oracle.MODE_STOCHASTIC):
            q_rm, _, scale = oracle.quantize2d(bits, mode, seed=0, tensor_id=0)
            deq = oracle.dequantize2d(q_rm, scale, *bits.shape)
            src = tensor.double().numpy()
            S = np.repeat(np.repeat(np.ldexp(1.0, scale.astype(np.int64) - 127), 32, 0), 32, 1)
            assert (np.abs(deq) <= 6 * S).all()
            assert (np.abs(src) <= 6 * S).all()                       # truncation-free: nothing clips
            step = np.where(np.abs(src) / S >= 4, 2.0, np.where(np.abs(src) / S >= 2, 1.0, 0.5)) * S
            bound = step / 2 if mode == oracle.MODE_NEAREST else step
            assert (np.abs(deq - src) <= bound).all()
            assert (np.signbit(deq) == np.signbit(src)).all()


def test_boundary_blocks_ignore_padding_and_pad_bytes_are_zero():
    # appendix "Boundary blocks": the scale of a partial block comes from its valid entries only.
    rng = np.random.default_rng(2)
    big = _random_bits(rng, 64, 64)
    big[40:, :] = 0x7F00          # huge values outside the 40x50 sub-matrix
    big[:, 50:] = 0x7F00
    sub = np.ascontiguousarray(big[:40, :50])
    q_rm, q_t, s = oracle.quantize2d(sub, oracle.MODE_NEAREST)
    assert q_rm.shape == (40, 25) and q_t.shape == (50, 20) and s.shape == (2, 2)
    codes, s_ref = _brute_force(sub, oracle.MODE_NEAREST, 0, 0)
    assert np.array_equal(s, s_ref)
    odd = np.ascontiguousarray(big[:33, :31])
    q_rm, q_t, _ = oracle.quantize2d(odd, oracle.MODE_NEAREST)
    assert (q_rm[:, -1] >> 4 == 0).all() and (q_t[:, -1] >> 4 == 0).all()   # the odd nibble is padding


def test_window_equals_slice_of_full_result():
    rng = np.random.default_rng(8)
    a = _random_bits(rng, 130, 200)
    q_rm, q_t, s = oracle.quantize2d(a, oracle.MODE_STOCHASTIC, seed=77, tensor_id=3)
    w_rm, w_t, ws = oracle.quantize2d(a, oracle.MODE_STOCHASTIC, seed=77, tensor_id=3, window=(1, 3, 2, 5))
    assert np.array_equal(ws, s[1:3, 2:5])
    assert np.array_equal(w_rm, q_rm[32:96, 32:80])
    assert np.array_equal(w_t, q_t[64:160, 16:48])


def test_empty_and_degenerate_inputs():
    for shape in [(0, 0), (0, 5), (7, 0)]:
        q_rm, q_t, s = oracle.quantize2d(np.zeros(shape, dtype=np.uint16))
        assert q_rm.size == 0 and q_t.size == 0
    q_rm, q_t, s = oracle.quantize2d(np.zeros((32, 32), dtype=np.uint16))
    assert not q_rm.any() and not q_t.any() and s[0, 0] == 0             # all-zero block: lowest scale
    bits = np.zeros((32, 32), dtype=np.uint16)
    bits[0, 0], bits[0, 1], bits[0, 2], bits[1, 0] = 0x7F80, 0xFF80, 0x7FC0, 0x3F80   # +Inf -Inf NaN 1.0
    q_rm, _, s = oracle.quantize2d(bits)
    n = _nibbles_rm(q_rm, 32)
    assert s[0, 0] == 125 and n[0, 0] == 0x7 and n[0, 1] == 0xF and n[0, 2] == 0 and n[1, 0] == 0x6


def test_stochastic_rounding_is_unbiased_over_ten_thousand_seeds():
    # E[roundS(x)] = x (Section 3.1): mean of the dequantized value over 10^4 seeds converges to the
    # input.  Per element: |mean - a| <= 4.5 * (step*S/2)/sqrt(n) + step*S/256  (a Bernoulli variable
    # scaled by the step has sd <= step/2; the second term is the floor(256 p) truncation).
    rng = np.random.default_rng(1)
    a = _random_bits(rng, 32, 32, scale_spread=False)
    n = 10_000
    acc = np.zeros((32, 32))
    for seed in range(n):
        q_rm, _, s = oracle.quantize2d(a, oracle.MODE_STOCHASTIC, seed=seed, tensor_id=0, want_t=False)
        acc += oracle.dequantize2d(q_rm, s, 32, 32)
    mean = acc / n
    S = 2.0 ** (int(s[0, 0]) - 127)
    src = np.array([[float(bf16_fraction(int(b))) for b in r] for r in a])
    ratio = np.abs(src) / S
    step = np.where(ratio >= 4, 2.0, np.where(ratio >= 2, 1.0, 0.5)) * S
    bound = 4.5 * (step / 2) / np.sqrt(n) + step / 256
    assert (np.abs(mean - src) <= bound).all()
    # and nearest rounding is visibly biased on the same data, so the test can tell the two apart
    q_rm, _, s = oracle.quantize2d(a, oracle.MODE_NEAREST, want_t=False)
    assert (np.abs(oracle.dequantize2d(q_rm, s, 32, 32) - src) > bound).mean() > 0.5
