"""CPU oracle for the fp4q hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Thin ctypes wrappers around ``fp4q_oracle.c`` (plain C, double precision, written
from the paper's definitions) plus the three linear-layer products of Section 3
("Application to linear layers") on dequantized values in float64.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It imports nothing from the CUDA package and shares no code,
table or constant with it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fp4q_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

BLOCK = 32
MODE_NEAREST = 0
MODE_STOCHASTIC = 1
FLAG_INDEX_TRANSPOSED = 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP if available). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, u64, u32, u8p = ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p
        L.orc_bf16_to_double.restype = ctypes.c_double
        L.orc_bf16_to_double.argtypes = [ctypes.c_uint16]
        L.orc_e2m1_value.restype = ctypes.c_double
        L.orc_e2m1_value.argtypes = [ctypes.c_int]
        L.orc_e4m3_value.restype = ctypes.c_double
        L.orc_e4m3_value.argtypes = [ctypes.c_int]
        L.orc_scale_exponent.restype = ctypes.c_int
        L.orc_scale_exponent.argtypes = [ctypes.c_double]
        L.orc_mxfp8_scale_exponent.restype = ctypes.c_int
        L.orc_mxfp8_scale_exponent.argtypes = [ctypes.c_double]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [ctypes.c_void_p] * 3
        L.orc_random_byte.restype = ctypes.c_uint
        L.orc_random_byte.argtypes = [u64, u32, u64]
        L.orc_round_nearest.restype = ctypes.c_int
        L.orc_round_nearest.argtypes = [ctypes.c_double]
        L.orc_round_stochastic.restype = ctypes.c_int
        L.orc_round_stochastic.argtypes = [ctypes.c_double, ctypes.c_uint]
        L.orc_round_nearest_e4m3.restype = ctypes.c_int
        L.orc_round_nearest_e4m3.argtypes = [ctypes.c_double]
        L.orc_quantize2d_window.restype = ctypes.c_int
        L.orc_quantize2d_window.argtypes = [u8p, i64, i64, i64, ctypes.c_int, u64, u32, u32,
                                            i64, i64, i64, i64, u8p, i64, u8p, i64, u8p, i64]
        L.orc_dequantize2d.restype = None
        L.orc_dequantize2d.argtypes = [u8p, i64, u8p, i64, i64, i64, u8p, i64]
        L.orc_quantize2d_block.restype = ctypes.c_int
        L.orc_quantize2d_block.argtypes = [u8p, i64, i64, i64, ctypes.c_int, ctypes.c_int, u64, u32, u32, u8p, i64, u8p, i64,
                                           u8p, i64]
        L.orc_dequantize2d_block.restype = None
        L.orc_dequantize2d_block.argtypes = [u8p, i64, u8p, i64, ctypes.c_int, i64, i64, u8p, i64]
        L.orc_quantize1d.restype = ctypes.c_int
        L.orc_quantize1d.argtypes = [u8p, i64, i64, i64, ctypes.c_int, u64, u32, u32, u8p, i64, u8p, i64]
        L.orc_dequantize1d.restype = None
        L.orc_dequantize1d.argtypes = [u8p, i64, u8p, i64, i64, i64, u8p, i64]
        L.orc_mxfp8_quantize1d.restype = ctypes.c_int
        L.orc_mxfp8_quantize1d.argtypes = [u8p, i64, i64, i64, u8p, i64, u8p, i64]
        L.orc_mxfp8_dequantize.restype = None
        L.orc_mxfp8_dequantize.argtypes = [u8p, i64, u8p, i64, i64, i64, u8p, i64]
        L.orc_gemm_nt.restype = None
        L.orc_gemm_nt.argtypes = [u8p, u8p, u8p, i64, i64, i64]
        L.orc_num_threads.restype = ctypes.c_int
        L.orc_num_threads.argtypes = []
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _as_bf16_bits(x) -> np.ndarray:
    """Accept a uint16 array of BF16 bit patterns (2-D)."""
    a = np.ascontiguousarray(x)
    if a.dtype != np.uint16 or a.ndim != 2:
        raise TypeError("expected a 2-D uint16 array of BF16 bit patterns")
    return a


def bits_to_double(x_bits) -> np.ndarray:
    """BF16 bit patterns -> float64 values (exact)."""
    x = _as_bf16_bits(x_bits)
    return (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def e2m1_value(code: int) -> float:
    return float(lib().orc_e2m1_value(int(code)))


def e4m3_value(code: int) -> float:
    return float(lib().orc_e4m3_value(int(code)))


def scale_exponent(M: float) -> int:
    return int(lib().orc_scale_exponent(float(M)))


def mxfp8_scale_exponent(M: float) -> int:
    return int(lib().orc_mxfp8_scale_exponent(float(M)))


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def random_byte(seed: int, tensor_id: int, idx: int) -> int:
    return int(lib().orc_random_byte(seed, tensor_id, idx))


def round_nearest(v: float) -> int:
    return int(lib().orc_round_nearest(float(v)))


def round_stochastic(v: float, r8: int) -> int:
    return int(lib().orc_round_stochastic(float(v), int(r8)))


def round_nearest_e4m3(v: float) -> int:
    return int(lib().orc_round_nearest_e4m3(float(v)))


def quantize2d(x_bits, mode=MODE_NEAREST, seed=0, tensor_id=0, flags=0, window=None, want_t=True):
    """2D-block FP4 quantization of a BF16 matrix given as uint16 bit patterns.

    Returns (q_rm [rows, ceil(cols/2)], q_t [cols, ceil(rows/2)] or None, scale [Rt, Ct]) as uint8.
    ``window=(I0, I1, J0, J1)`` restricts the work to those block rows/columns; the outputs are then
    indexed from the window's origin while the rounding stream stays keyed on the full tensor.
    """
    x = _as_bf16_bits(x_bits)
    rows, cols = x.shape
    rt, ct = -(-rows // BLOCK), -(-cols // BLOCK)
    I0, I1, J0, J1 = (0, rt, 0, ct) if window is None else window
    wrows = max(min(I1 * BLOCK, rows) - I0 * BLOCK, 0)
    wcols = max(min(J1 * BLOCK, cols) - J0 * BLOCK, 0)
    q_rm = np.zeros((wrows, (wcols + 1) // 2), dtype=np.uint8)
    q_t = np.zeros((wcols, (wrows + 1) // 2), dtype=np.uint8) if want_t else None
    scale = np.zeros((max(I1 - I0, 0), max(J1 - J0, 0)), dtype=np.uint8)
    if rows and cols and wrows and wcols:
        rc = lib().orc_quantize2d_window(
            _ptr(x), rows, cols, cols, mode, seed, tensor_id, flags, I0, I1, J0, J1,
            _ptr(q_rm), q_rm.shape[1], _ptr(q_t) if want_t else None, q_t.shape[1] if want_t else 0,
            _ptr(scale), scale.shape[1])
        if rc != 0:
            raise ValueError("orc_quantize2d_window rejected its arguments")
    return q_rm, q_t, scale


def dequantize2d(q_rm, scale, rows, cols):
    """Dequantized float64 matrix S * value(code) from the row-major payload."""
    q = np.ascontiguousarray(q_rm, dtype=np.uint8)
    s = np.ascontiguousarray(scale, dtype=np.uint8)
    out = np.zeros((rows, cols), dtype=np.float64)
    if rows and cols:
        lib().orc_dequantize2d(_ptr(q), q.shape[1], _ptr(s), s.shape[1], rows, cols, _ptr(out), cols)
    return out


def quantize2d_block(x_bits, block, mode=MODE_NEAREST, seed=0, tensor_id=0, flags=0, want_t=True):
    """The 2D scheme with b x b blocks (block-size study, Table 4).  Returns (q_rm, q_t or None,
    scale [ceil(rows/b), ceil(cols/b)]) as uint8."""
    x = _as_bf16_bits(x_bits)
    rows, cols = x.shape
    q_rm = np.zeros((rows, (cols + 1) // 2), dtype=np.uint8)
    q_t = np.zeros((cols, (rows + 1) // 2), dtype=np.uint8) if want_t else None
    scale = np.zeros((-(-rows // block), -(-cols // block)), dtype=np.uint8)
    if rows and cols:
        rc = lib().orc_quantize2d_block(_ptr(x), rows, cols, cols, int(block), int(mode), seed, tensor_id, flags,
                                        _ptr(q_rm), q_rm.shape[1], _ptr(q_t) if want_t else None,
                                        q_t.shape[1] if want_t else 0, _ptr(scale), scale.shape[1])
        if rc != 0:
            raise ValueError("orc_quantize2d_block rejected its arguments")
    return q_rm, q_t, scale


def dequantize2d_block(q_rm, scale, block, rows, cols):
    q = np.ascontiguousarray(q_rm, dtype=np.uint8)
    s = np.ascontiguousarray(scale, dtype=np.uint8)
    out = np.zeros((rows, cols), dtype=np.float64)
    if rows and cols:
        lib().orc_dequantize2d_block(_ptr(q), q.shape[1], _ptr(s), s.shape[1], int(block), rows, cols, _ptr(out), cols)
    return out


def quantize1d(x_bits, mode=MODE_NEAREST, seed=0, tensor_id=0, flags=0):
    """1D-block (1 x 32) FP4 quantization along the rows of a BF16 matrix (the paper's activation layout).
    Returns (q [rows, ceil(cols/2)], scale [rows, ceil(cols/32)]) as uint8."""
    x = _as_bf16_bits(x_bits)
    rows, cols = x.shape
    q = np.zeros((rows, (cols + 1) // 2), dtype=np.uint8)
    s = np.zeros((rows, -(-cols // BLOCK)), dtype=np.uint8)
    if rows and cols:
        rc = lib().orc_quantize1d(_ptr(x), rows, cols, cols, int(mode), seed, tensor_id, flags,
                                  _ptr(q), q.shape[1], _ptr(s), s.shape[1])
        if rc != 0:
            raise ValueError("orc_quantize1d rejected its arguments")
    return q, s


def quantize1d_t(x_bits, mode=MODE_NEAREST, seed=0, tensor_id=0):
    """The same encoding of the transpose (blocks along the rows of x, i.e. along the token axis when x is an
    activation [tokens, channels]); the rounding stream stays keyed on the element's index in x."""
    x = _as_bf16_bits(x_bits)
    return quantize1d(np.ascontiguousarray(x.T), mode, seed, tensor_id, FLAG_INDEX_TRANSPOSED)


def dequantize1d(q, scale, rows, cols):
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s = np.ascontiguousarray(scale, dtype=np.uint8)
    out = np.zeros((rows, cols), dtype=np.float64)
    if rows and cols:
        lib().orc_dequantize1d(_ptr(q), q.shape[1], _ptr(s), s.shape[1], rows, cols, _ptr(out), cols)
    return out


def transposition_diagnostic(x_bits):
    """Figure 1 (c), (d) of the paper on one tensor, nearest rounding: per element the difference of the scale
    exponents the element gets when the tensor is quantized as stored and when its transpose is quantized, and
    the relative Frobenius deviation between the two dequantized tensors - for 1D blocks and for 2D blocks.
    Returns a dict with the two exponent-difference maps and the two deviations."""
    x = _as_bf16_bits(x_bits)
    rows, cols = x.shape
    ref = bits_to_double(x)
    q1, s1 = quantize1d(x)
    q1t, s1t = quantize1d(np.ascontiguousarray(x.T))
    e_fwd = np.repeat(s1.astype(np.int32), BLOCK, axis=1)[:, :cols]
    e_bwd = np.repeat(s1t.astype(np.int32), BLOCK, axis=1)[:, :rows].T
    d1 = dequantize1d(q1, s1, rows, cols)
    d1t = dequantize1d(q1t, s1t, cols, rows).T
    q2, _, s2 = quantize2d(x, want_t=False)
    q2t, _, s2t = quantize2d(np.ascontiguousarray(x.T), want_t=False)
    f_fwd = np.repeat(np.repeat(s2.astype(np.int32), BLOCK, axis=0), BLOCK, axis=1)[:rows, :cols]
    f_bwd = np.repeat(np.repeat(s2t.astype(np.int32), BLOCK, axis=0), BLOCK, axis=1)[:cols, :rows].T
    d2 = dequantize2d(q2, s2, rows, cols)
    d2t = dequantize2d(q2t, s2t, cols, rows).T
    nrm = np.linalg.norm(ref)
    return {"scale_exponent_difference_1d": e_fwd - e_bwd, "scale_exponent_difference_2d": f_fwd - f_bwd,
            "deviation_1d": np.linalg.norm(d1 - d1t) / nrm, "deviation_2d": np.linalg.norm(d2 - d2t) / nrm}


def mxfp8_quantize1d(x_bits):
    """MXFP8 operand: E4M3 payload [rows, cols] and UE8M0 scales [rows, ceil(cols/32)]."""
    x = _as_bf16_bits(x_bits)
    rows, cols = x.shape
    q = np.zeros((rows, cols), dtype=np.uint8)
    s = np.zeros((rows, -(-cols // BLOCK)), dtype=np.uint8)
    if rows and cols:
        rc = lib().orc_mxfp8_quantize1d(_ptr(x), rows, cols, cols, _ptr(q), cols, _ptr(s), s.shape[1])
        if rc != 0:
            raise ValueError("orc_mxfp8_quantize1d rejected its arguments")
    return q, s


def mxfp8_quantize1d_t(x_bits):
    """MXFP8 operand of the transpose (the backward products of an MXFP8 projection contract over the other axis;
    Section 3.2 names the format only, the reading is: same rule, blocks along the new contraction axis)."""
    x = _as_bf16_bits(x_bits)
    return mxfp8_quantize1d(np.ascontiguousarray(x.T))


def mxfp8_dequantize(q, scale):
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s = np.ascontiguousarray(scale, dtype=np.uint8)
    rows, cols = q.shape
    out = np.zeros((rows, cols), dtype=np.float64)
    if rows and cols:
        lib().orc_mxfp8_dequantize(_ptr(q), cols, _ptr(s), s.shape[1], rows, cols, _ptr(out), cols)
    return out


def gemm_nt_definition(A, B):
    """C = A @ B^T by the plain triple loop (double). For small cases."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    C = np.zeros((M, N), dtype=np.float64)
    if M and N:
        lib().orc_gemm_nt(_ptr(A), _ptr(B), _ptr(C), M, N, K)
    return C


# The three products of Section 3 ("Application to linear layers") on dequantized float64 operands.
# A library matmul serves as the contraction step; every product of two dequantized values is exact in
# float64 and the sum is correct to ~1e-16 relative.

def gemm_fwd(x_hat, w_hat):
    """Y[T,N] = X^[T,K] W^[N,K]^T."""
    return np.asarray(x_hat, dtype=np.float64) @ np.asarray(w_hat, dtype=np.float64).T


def gemm_dgrad(dy_hat, w_hat):
    """dX[T,K] = dY^[T,N] W^[N,K]."""
    return np.asarray(dy_hat, dtype=np.float64) @ np.asarray(w_hat, dtype=np.float64)


def gemm_wgrad(dy_hat, x_hat):
    """dW[N,K] = dY^[T,N]^T X^[T,K]."""
    return np.asarray(dy_hat, dtype=np.float64).T @ np.asarray(x_hat, dtype=np.float64)


def grouped(fn, a, b_stack, row_offsets):
    """Grouped (MoE) form: rows row_offsets[g]..row_offsets[g+1] of the token matrix belong to expert g.

    fn in {gemm_fwd, gemm_dgrad}: b_stack is the expert weight stack [E*N, K]; result has a's row count.
    """
    E = len(row_offsets) - 1
    n_per = b_stack.shape[0] // E
    outs = []
    for g in range(E):
        r0, r1 = int(row_offsets[g]), int(row_offsets[g + 1])
        outs.append(fn(a[r0:r1], b_stack[g * n_per:(g + 1) * n_per]))
    return np.concatenate(outs, axis=0) if outs else np.zeros((0, 0))


def grouped_wgrad(dy_hat, x_hat, row_offsets):
    """dW stack [E*N, K]: dW_g = dY^[rows of g]^T X^[rows of g]."""
    E = len(row_offsets) - 1
    outs = []
    for g in range(E):
        r0, r1 = int(row_offsets[g]), int(row_offsets[g + 1])
        outs.append(gemm_wgrad(dy_hat[r0:r1], x_hat[r0:r1]))
    return np.concatenate(outs, axis=0)


def bf16_round(a):
    """Round float64 values to the nearest BF16 (ties to even), returned as float64."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    # float64 -> float32 is itself a rounding; BF16 outputs are compared with a tolerance that covers it
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)
