"""Pins for the oracle's block-size variants (block-size study, Table 4: the same 2D scheme with b x b blocks):
brute force in exact rationals for b = 16 and 64, identity with the pinned 32 x 32 quantizer at b = 32, the scale of
a 64-block against the four 32-block scales, transposition invariance at every block size, and the trend the paper
reports (smaller blocks, smaller error)."""
import numpy as np
import pytest

import oracle
from paper_2607_24953_b200 import workloads
from tests.exact import E2M1_MAGNITUDES, bf16_fraction, nearest_even_code, pow2, scale_exponent_exact


def _random_bits(rng, rows, cols):
    x = rng.standard_normal((rows, cols)).astype(np.float32) * np.exp(rng.standard_normal((rows, 1)) * 2).astype(np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16)


def _nibbles(q, n):
    out = np.zeros((q.shape[0], n), dtype=np.uint8)
    out[:, 0::2] = (q & 0xF)[:, :(n + 1) // 2]
    out[:, 1::2] = (q >> 4)[:, :n // 2]
    return out


def _brute_force(bits, b, mode, seed, tid):
    rows, cols = bits.shape
    rt, ct = -(-rows // b), -(-cols // b)
    codes = np.zeros((rows, cols), dtype=np.uint8)
    scale = np.zeros((rt, ct), dtype=np.uint8)
    for I in range(rt):
        for J in range(ct):
            blk = [(i, j) for i in range(b * I, min(b * I + b, rows)) for j in range(b * J, min(b * J + b, cols))]
            M = max(abs(bf16_fraction(int(bits[i, j]))) for i, j in blk)
            e = scale_exponent_exact(M)
            scale[I, J] = e + 127
            for i, j in blk:
                v = abs(bf16_fraction(int(bits[i, j]))) / pow2(e)
                if mode == oracle.MODE_NEAREST:
                    mag = nearest_even_code(v)
                else:
                    idx = i * cols + j
                    out = oracle.philox4x32_10([(idx >> 4) & 0xFFFFFFFF, (idx >> 4) >> 32, tid, 0], [seed & 0xFFFFFFFF, seed >> 32])
                    r8 = (int(out[(idx >> 2) & 3]) >> (8 * (idx & 3))) & 0xFF
                    lo = max(c for c in range(8) if E2M1_MAGNITUDES[c] <= v)
                    if lo == 7:
                        mag = 7
                    else:
                        p = (v - E2M1_MAGNITUDES[lo]) / (E2M1_MAGNITUDES[lo + 1] - E2M1_MAGNITUDES[lo])
                        mag = lo + 1 if int(256 * p) + r8 >= 256 else lo
                codes[i, j] = ((int(bits[i, j]) >> 15) << 3) | mag
    return codes, scale


@pytest.mark.parametrize("b,shape", [(16, (32, 48)), (16, (17, 33)), (64, (64, 128)), (64, (70, 65)), (8, (16, 24))])
@pytest.mark.parametrize("mode", [oracle.MODE_NEAREST, oracle.MODE_STOCHASTIC])
def test_against_exact_brute_force(b, shape, mode):
    rng = np.random.default_rng(b * 1000 + shape[0])
    bits = _random_bits(rng, *shape)
    q_rm, q_t, scale = oracle.quantize2d_block(bits, b, mode, seed=77, tensor_id=3)
    codes, scale_ref = _brute_force(bits, b, mode, 77, 3)
    assert np.array_equal(scale, scale_ref)
    assert np.array_equal(_nibbles(q_rm, shape[1]), codes)
    assert np.array_equal(_nibbles(q_t, shape[0]), codes.T)


@pytest.mark.parametrize("mode", [oracle.MODE_NEAREST, oracle.MODE_STOCHASTIC])
def test_block_32_is_the_pinned_quantizer(mode):
    rng = np.random.default_rng(5)
    bits = _random_bits(rng, 100, 75)
    a = oracle.quantize2d_block(bits, 32, mode, seed=4, tensor_id=2)
    b = oracle.quantize2d(bits, mode, seed=4, tensor_id=2)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)


def test_scale_of_a_64_block_is_the_largest_of_its_four_32_blocks():
    # S is monotone in the block maximum, and the maximum of a 64-block is the largest of its quarters' maxima
    rng = np.random.default_rng(6)
    bits = _random_bits(rng, 192, 256)
    _, _, s64 = oracle.quantize2d_block(bits, 64, want_t=False)
    _, _, s32 = oracle.quantize2d(bits, want_t=False)
    pooled = s32.reshape(3, 2, 4, 2).max(axis=(1, 3))
    assert np.array_equal(s64, pooled)
    _, _, s16 = oracle.quantize2d_block(bits, 16, want_t=False)
    assert np.array_equal(s32, s16.reshape(6, 2, 8, 2).max(axis=(1, 3)))


@pytest.mark.parametrize("b", [16, 64])
def test_transposition_invariance_at_every_block_size(b):
    rng = np.random.default_rng(7)
    bits = _random_bits(rng, 96, 160)
    q_rm, q_t, s = oracle.quantize2d_block(bits, b)
    r_rm, r_t, rs = oracle.quantize2d_block(np.ascontiguousarray(bits.T), b)
    assert np.array_equal(s.T, rs) and np.array_equal(q_t, r_rm) and np.array_equal(q_rm, r_t)
    # stochastic rounding with the transposed index draws the same byte for the same element
    a = oracle.quantize2d_block(bits, b, oracle.MODE_STOCHASTIC, seed=3, tensor_id=1)
    c = oracle.quantize2d_block(np.ascontiguousarray(bits.T), b, oracle.MODE_STOCHASTIC, seed=3, tensor_id=1,
                                flags=oracle.FLAG_INDEX_TRANSPOSED)
    assert np.array_equal(a[1], c[0]) and np.array_equal(a[2].T, c[2])


def test_error_grows_with_the_block_size_and_nothing_clips():
    # Table 4's trend: a smaller block follows local magnitudes more closely.  On an activation with outlier
    # channels the relative error is ordered 16 <= 32 <= 64; no dequantized value exceeds 6 S and |error| <= S
    x = workloads.bf16_bits(workloads.activations_gauss_outliers(256, 512, seed=11))
    ref = oracle.bits_to_double(x)
    errs = []
    for b in (16, 32, 64):
        q, _, s = oracle.quantize2d_block(x, b, want_t=False)
        d = oracle.dequantize2d_block(q, s, b, 256, 512)
        S = np.repeat(np.repeat(np.ldexp(1.0, s.astype(np.int32) - 127), b, 0), b, 1)[:256, :512]
        assert (np.abs(d) <= 6 * S).all() and (np.abs(d - ref) <= S).all()
        errs.append(np.linalg.norm(d - ref) / np.linalg.norm(ref))
    assert errs[0] <= errs[1] <= errs[2] and errs[0] < errs[2]
