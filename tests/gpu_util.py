"""Helpers shared by the GPU parity tests (tests only)."""
import numpy as np
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads


def bits_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return workloads.bits_to_bf16(bits, device)


def gpu_quantize(x: torch.Tensor, mode, seed=0, tensor_id=0, flags=0, want_t=True):
    qt = binding.fp4q_quantize2d(x, mode=mode, seed=seed, tensor_id=tensor_id, flags=flags, want_t=want_t)
    torch.cuda.synchronize()
    return qt


def logical(qt: binding.QTensor):
    """Payload bytes of the logical extent and of the block padding, as numpy arrays."""
    rows, cols = qt.rows, qt.cols
    q_rm = qt.q_rm.cpu().numpy()
    q_t = qt.q_t.cpu().numpy() if qt.q_t is not None else None
    scale = qt.scale.cpu().numpy()[:, :max((cols + 31) // 32, 0)]
    return q_rm, q_t, scale


def assert_matches_oracle(x: torch.Tensor, mode, seed=0, tensor_id=0, flags=0, want_t=True):
    """Bit-exact comparison of the CUDA quantizer with the oracle on the same bytes."""
    rows, cols = x.shape
    qt = gpu_quantize(x, mode, seed, tensor_id, flags, want_t)
    g_rm, g_t, g_s = logical(qt)
    bits = workloads.bf16_bits(x)
    o_rm, o_t, o_s = oracle.quantize2d(bits, mode, seed, tensor_id, flags, want_t=want_t)
    assert np.array_equal(g_s, o_s), "scales differ"
    w = (cols + 1) // 2
    assert np.array_equal(g_rm[:, :w], o_rm), "row-major payload differs"
    pad_to = (cols + 31) // 32 * 16
    assert not g_rm[:, w:pad_to].any(), "row-major block padding is not zero"
    if want_t:
        h = (rows + 1) // 2
        assert np.array_equal(g_t[:, :h], o_t), "transposed payload differs"
        assert not g_t[:, h:(rows + 31) // 32 * 16].any(), "transposed block padding is not zero"
    return qt


def dequant_from_gpu(qt: binding.QTensor) -> np.ndarray:
    """Dequantize a GPU result with the oracle's decoder (row-major payload)."""
    g_rm, _, g_s = logical(qt)
    return oracle.dequantize2d(np.ascontiguousarray(g_rm[:, :(qt.cols + 1) // 2]), np.ascontiguousarray(g_s),
                               qt.rows, qt.cols)


def check_gemm(got: torch.Tensor, ref: np.ndarray, what=""):
    """The GEMM tolerance of the build target: relative Frobenius error <= 1e-3 and, per output row,
    max |G - O| <= 1e-2 * ||O_row||_inf.  BF16 outputs are compared with the oracle rounded to BF16."""
    g = got.double().cpu().numpy()
    if got.dtype == torch.bfloat16:
        ref = oracle.bf16_round(ref)
    assert g.shape == ref.shape, (g.shape, ref.shape)
    denom = np.linalg.norm(ref)
    rel = np.linalg.norm(g - ref) / denom if denom > 0 else np.abs(g).max()
    assert rel <= 1e-3, "%s: relative Frobenius error %.3e" % (what, rel)
    row_inf = np.abs(ref).max(axis=1, keepdims=True)
    assert (np.abs(g - ref) <= 1e-2 * row_inf + 1e-300).all(), "%s: per-row max-abs bound violated" % what
    return rel


class HostQ:
    """Host copy of a 2D-block-quantized tensor; rows and columns are decoded with the oracle's decoder and
    value table (row-major payload for rows, transposed payload for columns, so both layouts are exercised)."""

    def __init__(self, qt: binding.QTensor):
        self.rows, self.cols = qt.rows, qt.cols
        self.q_rm = qt.q_rm.cpu().numpy()
        self.q_t = qt.q_t.cpu().numpy() if qt.q_t is not None else None
        self.scale = qt.scale.cpu().numpy()
        self._values = np.array([oracle.e2m1_value(k) for k in range(16)])

    def row_range(self, r0: int, r1: int) -> np.ndarray:
        """Dequantized rows r0..r1 (r0 a multiple of 32)."""
        assert r0 % 32 == 0
        n = r1 - r0
        if n <= 0:
            return np.zeros((0, self.cols))
        q = np.ascontiguousarray(self.q_rm[r0:r1, :(self.cols + 1) // 2])
        s = np.ascontiguousarray(self.scale[r0 // 32:(r1 + 31) // 32, :max((self.cols + 31) // 32, 1)])
        return oracle.dequantize2d(q, s, n, self.cols)

    def take_rows(self, rows) -> np.ndarray:
        out = np.empty((len(rows), self.cols))
        for i, r in enumerate(rows):
            b = int(r) // 32 * 32
            out[i] = self.row_range(b, min(b + 32, self.rows))[int(r) - b]
        return out

    def take_cols(self, cols, r0: int = 0, r1: int = None) -> np.ndarray:
        """Dequantized columns (as an array [r1 - r0, len(cols)]) decoded from the transposed payload."""
        r1 = self.rows if r1 is None else r1
        assert r0 % 32 == 0
        out = np.empty((r1 - r0, len(cols)))
        for i, c in enumerate(cols):
            q = self.q_t[int(c), r0 // 2:(r1 + 1) // 2]
            codes = np.empty(2 * q.size, dtype=np.uint8)
            codes[0::2] = q & 0xF
            codes[1::2] = q >> 4
            e = np.repeat(self.scale[r0 // 32:(r1 + 31) // 32, int(c) // 32].astype(np.int64), 32)[:r1 - r0]
            out[:, i] = self._values[codes[:r1 - r0]] * np.ldexp(1.0, e - 127)
        return out


def assert_windows_match_oracle(x: torch.Tensor, qt: binding.QTensor, block_rows, mode, seed, tensor_id):
    """Bit-exact comparison of whole block rows (32 rows, every column) of a large quantized tensor with the
    oracle, which is run on a window of the full tensor (the rounding stream stays keyed on the global index)."""
    bits = workloads.bf16_bits(x)
    rows, cols = bits.shape
    ct = (cols + 31) // 32
    for I in block_rows:
        I = int(I)
        o_rm, o_t, o_s = oracle.quantize2d(bits, mode, seed, tensor_id, window=(I, I + 1, 0, ct))
        n = o_rm.shape[0]
        g_rm = qt.q_rm[32 * I:32 * I + n, :(cols + 1) // 2].cpu().numpy()
        g_t = qt.q_t[:cols, 16 * I:16 * I + (n + 1) // 2].cpu().numpy()
        g_s = qt.scale[I, :ct].cpu().numpy()
        assert np.array_equal(g_s, o_s[0]), ("scale", I)
        assert np.array_equal(g_rm, o_rm), ("q_rm", I)
        assert np.array_equal(g_t, o_t), ("q_t", I)
