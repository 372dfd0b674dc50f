"""Pins for the oracle's number formats (E2M1, E4M3) and for Philox4x32-10."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from tests.exact import E2M1_MAGNITUDES

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_e2m1_table_matches_format_definition():
    # Section 2: E2M1. Magnitudes of codes 0..7 and their negatives for codes 8..15.
    for c in range(8):
        assert Fraction(oracle.e2m1_value(c)) == E2M1_MAGNITUDES[c]
        assert Fraction(oracle.e2m1_value(c + 8)) == -E2M1_MAGNITUDES[c]
    assert np.signbit(oracle.e2m1_value(8))          # -0 keeps its sign
    assert oracle.e2m1_value(7) == 6.0 and oracle.e2m1_value(15) == -6.0   # Q_p, Q_n of Section 3.1


def test_e2m1_table_matches_cuda_fp4_library(library_pins):
    for c in range(16):
        assert oracle.e2m1_value(c) == library_pins.pin_fp4_decode(c)


def test_e4m3_table_matches_torch_and_cuda_fp8(library_pins):
    import torch
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for c in range(256):
        v = oracle.e4m3_value(c)
        if c in (0x7F, 0xFF):
            assert np.isnan(v) and np.isnan(ref[c])
        else:
            assert v == ref[c] == library_pins.pin_e4m3_decode(c)
    assert oracle.e4m3_value(0x7E) == 448.0


def _read_kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([int(t, 16) for t in line.split()])
    return rows


def test_philox_known_answers():
    for r in _read_kat():
        out = oracle.philox4x32_10(r[0:4], r[4:6])
        assert list(map(int, out)) == r[6:10]


def test_philox_matches_two_libraries(library_pins):
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = rng.integers(0, 2 ** 32, size=4, dtype=np.uint64).astype(np.uint32)
        key = rng.integers(0, 2 ** 32, size=2, dtype=np.uint64).astype(np.uint32)
        mine = oracle.philox4x32_10(ctr, key)
        cu = np.zeros(4, dtype=np.uint32)
        library_pins.pin_philox_curand(ctr.ctypes.data, key.ctypes.data, cu.ctypes.data)
        at = np.zeros(4, dtype=np.uint32)
        seed = int(key[0]) | (int(key[1]) << 32)
        offset = int(ctr[0]) | (int(ctr[1]) << 32)
        subseq = int(ctr[2]) | (int(ctr[3]) << 32)
        library_pins.pin_philox_aten(seed, subseq, offset, at.ctypes.data)
        assert list(mine) == list(cu) == list(at)


def test_random_byte_indexing():
    # 16 consecutive element indices share one Philox block; byte b of word w belongs to index 4w+b.
    seed, tid = 0x0123456789ABCDEF, 77
    for blk in (0, 1, 5, 2 ** 32 + 3):
        out = oracle.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, tid, 0], [seed & 0xFFFFFFFF, seed >> 32])
        for k in range(16):
            expect = (int(out[k // 4]) >> (8 * (k % 4))) & 0xFF
            assert oracle.random_byte(seed, tid, 16 * blk + k) == expect


def test_random_bytes_uniform_chi_square():
    n = 1 << 16
    counts = np.zeros(256)
    for i in range(n):
        counts[oracle.random_byte(12345, 3, i)] += 1
    chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
    assert chi2 < 340.0    # 255 dof: mean 255, sd 22.6; 340 is ~3.8 sd


def test_table1_storage_arithmetic():
    # Table 1 counts payload bits only; the oracle's payload sizes (4 bits per 2D-FP4 element, 8 per
    # MXFP8 element) reproduce the printed megabytes and the ~3.56x ideal throughput.
    rows = {}
    with open(os.path.join(GOLDEN, "table1_weight_storage.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                t = line.split()
                rows[t[0]] = t[1:]
    x = np.zeros((64, 64), dtype=np.uint16)
    q_rm, _, _ = oracle.quantize2d(x)
    q8, _ = oracle.mxfp8_quantize1d(x)
    bits = {"4": q_rm.size * 8 / x.size, "8": q8.size * 8 / x.size}
    assert bits == {"4": 4.0, "8": 8.0}
    for name in ("qk_linear", "other_attn_linear", "mlp_linear"):
        bf16_mb, method_mb, b = float(rows[name][0]), float(rows[name][1]), rows[name][2]
        assert abs(bf16_mb * bits[b] / 16.0 - method_mb) <= 0.06
    total = sum(float(rows[n][1]) for n in ("qk_linear", "other_attn_linear", "mlp_linear"))
    assert abs(total - float(rows["transformer_linear"][1])) <= 0.11
    f8 = float(rows["ideal_linear_speedup"][2])
    assert abs(1.0 / (f8 / 2 + (1 - f8) / 4) - float(rows["ideal_linear_speedup"][0])) < 0.01
