"""Thin Python binding of libfp4q.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/fp4q.h) and does nothing
but turn torch tensors into device pointers, sizes and leading dimensions.  All arithmetic runs in
the CUDA kernels of the library.  There is no CPU fallback: if the library is missing or the
tensors are not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FP4Q_LIB") or os.path.join(_HERE, "libfp4q.so")   # FP4Q_LIB: load another build of the library

ROUND_NEAREST = 0
ROUND_STOCHASTIC = 1
OUT_BF16 = 0
OUT_F32 = 1
INDEX_TRANSPOSED = 1
BLOCK_16 = 2   # fp4q_quantize2d flags: 16 x 16 or 64 x 64 blocks instead of 32 x 32 (block-size study)
BLOCK_64 = 4

EXPORTS = ["fp4q_quantize2d", "fp4q_gemm_fwd", "fp4q_gemm_dgrad", "fp4q_gemm_wgrad",
           "fp4q_mxfp8_quantize1d", "fp4q_mxfp8_qk", "fp4q_workspace_bytes", "fp4q_workspace_status",
           "fp4q_status_string", "fp4q_version", "fp4q_gemm_fwd_static_workspace", "fp4q_workspace_set_wait_limit",
           "fp4q_debug_withhold_load", "fp4q_quantize1d", "fp4q_quantize1d_t", "fp4q_gemm_fwd_act1d", "fp4q_gemm_wgrad_act1d",
           "fp4q_mxfp8_quantize1d_t", "fp4q_mxfp8_gemm", "fp4q_gemm_fwd_quantized", "fp4q_gemm_dgrad_quantized",
           "fp4q_gemm_fwd_b16", "fp4q_gemm_dgrad_b16", "fp4q_gemm_wgrad_b16", "fp4q_quantize2d_multi"]


class Fp4qError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, status_string(status)))


class _CTensor(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("q_rm", ctypes.c_void_p), ("ld_rm", ctypes.c_int64),
                ("q_t", ctypes.c_void_p), ("ld_t", ctypes.c_int64),
                ("scale", ctypes.c_void_p), ("ld_s", ctypes.c_int64)]


class _CQuantJob(ctypes.Structure):
    _fields_ = [("x_bf16", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("ld_x", ctypes.c_int64),
                ("out", ctypes.POINTER(_CTensor)), ("tensor_id", ctypes.c_uint32), ("flags", ctypes.c_uint32)]


class _CGroups(ctypes.Structure):
    _fields_ = [("n_groups", ctypes.c_int32), ("row_alignment", ctypes.c_int32), ("row_offsets", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libfp4q.so (built in-tree by paper_2607_24953_b200.build). Fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libfp4q.so is not built: run `python -m paper_2607_24953_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i64, u64, u32, vp, ci = ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_int
        L.fp4q_quantize2d.restype = ci
        L.fp4q_quantize2d.argtypes = [vp, i64, i64, i64, ctypes.POINTER(_CTensor), ci, u64, u32, u32, vp]
        L.fp4q_mxfp8_quantize1d.restype = ci
        L.fp4q_mxfp8_quantize1d.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, vp]
        L.fp4q_workspace_bytes.restype = ctypes.c_size_t
        L.fp4q_workspace_bytes.argtypes = []
        L.fp4q_workspace_status.restype = ci
        L.fp4q_workspace_status.argtypes = [vp, vp]
        L.fp4q_workspace_set_wait_limit.restype = ci
        L.fp4q_workspace_set_wait_limit.argtypes = [vp, u32, vp]
        L.fp4q_debug_withhold_load.restype = ci
        L.fp4q_debug_withhold_load.argtypes = [vp, u32, vp]
        L.fp4q_status_string.restype = ctypes.c_char_p
        L.fp4q_status_string.argtypes = [ci]
        L.fp4q_version.restype = ci
        L.fp4q_version.argtypes = []
        gemm_args = [ctypes.POINTER(_CTensor), ctypes.POINTER(_CTensor), vp, i64, ci, ctypes.POINTER(_CGroups),
                     vp, ctypes.c_size_t, vp]
        L.fp4q_gemm_fwd.restype = ci
        L.fp4q_gemm_fwd.argtypes = gemm_args
        L.fp4q_gemm_dgrad.restype = ci
        L.fp4q_gemm_dgrad.argtypes = gemm_args
        L.fp4q_gemm_wgrad.restype = ci
        L.fp4q_gemm_wgrad.argtypes = gemm_args[:5] + [ci] + gemm_args[5:]
        L.fp4q_mxfp8_qk.restype = ci
        L.fp4q_mxfp8_qk.argtypes = [vp, i64, vp, i64, i64, i64, vp, vp, vp, vp, i64, i64, i64, vp, vp, i64,
                                    ci, vp, ctypes.c_size_t, vp]
        L.fp4q_gemm_fwd_static_workspace.restype = ci
        L.fp4q_gemm_fwd_static_workspace.argtypes = [ctypes.POINTER(_CTensor), ctypes.POINTER(_CTensor), vp, i64,
                                                     ci, vp, vp]
        L.fp4q_quantize1d.restype = ci
        L.fp4q_quantize1d.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, ci, u64, u32, vp]
        L.fp4q_quantize1d_t.restype = ci
        L.fp4q_quantize1d_t.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, vp]
        L.fp4q_gemm_fwd_act1d.restype = ci
        L.fp4q_gemm_fwd_act1d.argtypes = [vp, i64, vp, i64, i64, vp, vp, i64, ci, vp, ctypes.c_size_t, vp]
        L.fp4q_gemm_wgrad_act1d.restype = ci
        L.fp4q_gemm_wgrad_act1d.argtypes = [vp, vp, i64, vp, i64, i64, vp, i64, ci, ci, vp, ctypes.c_size_t, vp]
        L.fp4q_mxfp8_quantize1d_t.restype = ci
        L.fp4q_mxfp8_quantize1d_t.argtypes = [vp, i64, i64, i64, vp, i64, vp, i64, vp]
        L.fp4q_mxfp8_gemm.restype = ci
        L.fp4q_mxfp8_gemm.argtypes = [vp, i64, vp, i64, i64, vp, i64, vp, i64, i64, i64, vp, i64, ci, vp,
                                      ctypes.c_size_t, vp]
        L.fp4q_gemm_dgrad_quantized.restype = ci
        L.fp4q_gemm_dgrad_quantized.argtypes = [vp, vp, vp, ci, u64, u32, vp, vp, ctypes.c_size_t, vp]
        L.fp4q_gemm_fwd_quantized.restype = ci
        L.fp4q_gemm_fwd_quantized.argtypes = [ctypes.POINTER(_CTensor), ctypes.POINTER(_CTensor),
                                              ctypes.POINTER(_CTensor), ci, u64, u32, vp, vp, ctypes.c_size_t, vp]
        L.fp4q_quantize2d_multi.restype = ci
        L.fp4q_quantize2d_multi.argtypes = [ctypes.POINTER(_CQuantJob), ctypes.c_int32, ci, u64, vp]
        b16_args = [ctypes.POINTER(_CTensor), ctypes.POINTER(_CTensor), vp, i64, ci, vp, ctypes.c_size_t, vp]
        L.fp4q_gemm_fwd_b16.restype = ci
        L.fp4q_gemm_fwd_b16.argtypes = b16_args
        L.fp4q_gemm_dgrad_b16.restype = ci
        L.fp4q_gemm_dgrad_b16.argtypes = b16_args
        L.fp4q_gemm_wgrad_b16.restype = ci
        L.fp4q_gemm_wgrad_b16.argtypes = b16_args[:5] + [ci] + b16_args[5:]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().fp4q_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise Fp4qError(status, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError("%s must live on a CUDA device (there is no CPU path)" % name)
    return t


@dataclass
class QTensor:
    """Device buffers of a 2D-block-quantized tensor (fp4q_tensor of include/fp4q.h)."""
    rows: int
    cols: int
    q_rm: torch.Tensor               # uint8 [rows, ld_rm]
    q_t: Optional[torch.Tensor]      # uint8 [cols, ld_t] or None
    scale: torch.Tensor              # uint8 [ceil(rows/32), ld_s] ([ceil(rows/16), ld_s] after BLOCK_16)
    scale_granularity: int = 32      # 16 only for tensors quantized with BLOCK_16, which only the *_b16 products take

    def c_struct(self, granularity: int = 32) -> _CTensor:
        """granularity: the scale granularity the callee expects (0 = any: the quantizer's own output)."""
        if granularity and self.scale_granularity != granularity:
            raise ValueError("this call takes tensors quantized in %d x %d blocks (scale matrix of that granularity); got %d"
                             % (granularity, granularity, self.scale_granularity))
        return _CTensor(self.rows, self.cols,
                        self.q_rm.data_ptr(), self.q_rm.stride(0),
                        self.q_t.data_ptr() if self.q_t is not None else None,
                        self.q_t.stride(0) if self.q_t is not None else 0,
                        self.scale.data_ptr(), self.scale.stride(0))


def _pad16(n: int) -> int:
    return (n + 15) // 16 * 16


def alloc_qtensor(rows: int, cols: int, device, want_t: bool = True, scale_granularity: int = 32) -> QTensor:
    """Allocate the output buffers of fp4q_quantize2d with the leading dimensions the ABI asks for."""
    ld_rm = max(_pad16((cols + 31) // 32 * 16), 16)
    ld_t = max(_pad16((rows + 31) // 32 * 16), 16)
    q_rm = torch.empty((rows, ld_rm), dtype=torch.uint8, device=device)
    q_t = torch.empty((cols, ld_t), dtype=torch.uint8, device=device) if want_t else None
    g = scale_granularity
    scale = torch.empty(((rows + g - 1) // g, max((cols + g - 1) // g, 1)), dtype=torch.uint8, device=device)
    return QTensor(rows, cols, q_rm, q_t, scale, g)


def fp4q_quantize2d(x: torch.Tensor, out: Optional[QTensor] = None, mode: int = ROUND_NEAREST, seed: int = 0,
                    tensor_id: int = 0, flags: int = 0, want_t: bool = True, stream=None) -> QTensor:
    """x: BF16 [rows, cols] on the GPU, unit stride along columns. Returns (and fills) a QTensor."""
    _dev(x, "x")
    if x.dtype != torch.bfloat16 or x.dim() != 2 or (x.numel() and x.stride(1) != 1):
        raise ValueError("x must be a 2-D BF16 tensor with contiguous rows")
    rows, cols = x.shape
    if out is None:
        out = alloc_qtensor(rows, cols, x.device, want_t, 16 if flags & BLOCK_16 else 32)
    cs = out.c_struct(granularity=0)
    st = lib().fp4q_quantize2d(x.data_ptr(), rows, cols, x.stride(0) if rows else cols, ctypes.byref(cs),
                               mode, seed, tensor_id, flags, _stream(stream))
    _check(st, "fp4q_quantize2d")
    return out


def fp4q_quantize2d_multi(xs, outs=None, mode: int = ROUND_NEAREST, seed: int = 0, tensor_ids=None, flags: int = 0,
                          want_t: bool = True, stream=None):
    """fp4q_quantize2d of several independent BF16 tensors by one call (chained launches in one stream).  xs: list of 2-D BF16 device tensors; outs: matching
    list of QTensor (allocated when None); tensor_ids: one rounding-stream id per tensor (default 0, 1, ...)."""
    n = len(xs)
    if outs is None:
        outs = [alloc_qtensor(x.shape[0], x.shape[1], x.device, want_t) for x in xs]
    if tensor_ids is None:
        tensor_ids = list(range(n))
    structs = [o.c_struct() for o in outs]                    # kept alive until the call returns
    jobs = (_CQuantJob * max(n, 1))()
    for j, x in enumerate(xs):
        _dev(x, "xs[%d]" % j)
        if x.dtype != torch.bfloat16 or x.dim() != 2 or (x.numel() and x.stride(1) != 1):
            raise ValueError("every input must be a 2-D BF16 tensor with contiguous rows")
        jobs[j] = _CQuantJob(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0) if x.shape[0] else x.shape[1],
                             ctypes.pointer(structs[j]), int(tensor_ids[j]), flags)
    _check(lib().fp4q_quantize2d_multi(jobs, n, mode, seed, _stream(stream)), "fp4q_quantize2d_multi")
    return outs


def fp4q_mxfp8_quantize1d(x: torch.Tensor, stream=None):
    """x: BF16 [rows, cols]. Returns (q uint8 [rows, ld_q], scale uint8 [rows, ceil(cols/32)])."""
    _dev(x, "x")
    if x.dtype != torch.bfloat16 or x.dim() != 2 or (x.numel() and x.stride(1) != 1):
        raise ValueError("x must be a 2-D BF16 tensor with contiguous rows")
    rows, cols = x.shape
    ld_q = max((cols + 31) // 32 * 32, 32)
    q = torch.empty((rows, ld_q), dtype=torch.uint8, device=x.device)
    scale = torch.empty((rows, max((cols + 31) // 32, 1)), dtype=torch.uint8, device=x.device)
    st = lib().fp4q_mxfp8_quantize1d(x.data_ptr(), rows, cols, x.stride(0) if rows else cols, q.data_ptr(), ld_q,
                                     scale.data_ptr(), scale.stride(0), _stream(stream))
    _check(st, "fp4q_mxfp8_quantize1d")
    return q, scale


def fp4q_quantize1d(x: torch.Tensor, mode: int = ROUND_NEAREST, seed: int = 0, tensor_id: int = 0, stream=None):
    """1D-block FP4 of x (blocks along its rows).  Returns (q uint8 [rows, ld_q], scale uint8 [rows, ceil(cols/32)])."""
    _dev(x, "x")
    if x.dtype != torch.bfloat16 or x.dim() != 2 or (x.numel() and x.stride(1) != 1):
        raise ValueError("x must be a 2-D BF16 tensor with contiguous rows")
    rows, cols = x.shape
    ld_q = max(_pad16((cols + 31) // 32 * 16), 16)
    q = torch.empty((rows, ld_q), dtype=torch.uint8, device=x.device)
    scale = torch.empty((rows, max((cols + 31) // 32, 1)), dtype=torch.uint8, device=x.device)
    st = lib().fp4q_quantize1d(x.data_ptr(), rows, cols, x.stride(0) if rows else cols, q.data_ptr(), ld_q,
                               scale.data_ptr(), scale.stride(0), mode, seed, tensor_id, _stream(stream))
    _check(st, "fp4q_quantize1d")
    return q, scale


def fp4q_quantize1d_t(x: torch.Tensor, stream=None):
    """1D-block FP4 of x^T (blocks along the rows of x), nearest rounding.  Returns (q [cols, ld_q], scale [cols, ceil(rows/32)])."""
    _dev(x, "x")
    if x.dtype != torch.bfloat16 or x.dim() != 2 or (x.numel() and x.stride(1) != 1):
        raise ValueError("x must be a 2-D BF16 tensor with contiguous rows")
    rows, cols = x.shape
    ld_q = max(_pad16((rows + 31) // 32 * 16), 16)
    q = torch.empty((cols, ld_q), dtype=torch.uint8, device=x.device)
    scale = torch.empty((cols, max((rows + 31) // 32, 1)), dtype=torch.uint8, device=x.device)
    st = lib().fp4q_quantize1d_t(x.data_ptr(), rows, cols, x.stride(0) if rows else cols, q.data_ptr(), ld_q,
                                 scale.data_ptr(), scale.stride(0), _stream(stream))
    _check(st, "fp4q_quantize1d_t")
    return q, scale


def fp4q_mxfp8_quantize1d_t(x: torch.Tensor, stream=None):
    """MXFP8 encoding of x^T.  x: BF16 [rows, cols].  Returns (q uint8 [cols, ld_q], scale uint8 [cols, ceil(rows/32)])."""
    _dev(x, "x")
    if x.dtype != torch.bfloat16 or x.dim() != 2 or (x.numel() and x.stride(1) != 1):
        raise ValueError("x must be a 2-D BF16 tensor with contiguous rows")
    rows, cols = x.shape
    ld_q = max((rows + 31) // 32 * 32, 32)
    q = torch.empty((cols, ld_q), dtype=torch.uint8, device=x.device)
    scale = torch.empty((cols, max((rows + 31) // 32, 1)), dtype=torch.uint8, device=x.device)
    st = lib().fp4q_mxfp8_quantize1d_t(x.data_ptr(), rows, cols, x.stride(0) if rows else cols, q.data_ptr(), ld_q,
                                       scale.data_ptr(), scale.stride(0), _stream(stream))
    _check(st, "fp4q_mxfp8_quantize1d_t")
    return q, scale


def fp4q_mxfp8_gemm(aq, a_s, bq, b_s, M: int, N: int, Kdim: int, dt: int = OUT_BF16, ws=None, stream=None):
    """C[M,N] = A^ B^^T on MXFP8 operands (rows along the contraction axis) from the two MXFP8 quantizers."""
    dev = aq.device
    per16 = 8 if dt == OUT_BF16 else 4
    ldc = max((N + per16 - 1) // per16 * per16, per16)
    out = torch.empty((M, ldc), dtype=_out_dtype(dt), device=dev)[:, :N]
    if ws is None:
        ws = alloc_workspace(dev)
    st = lib().fp4q_mxfp8_gemm(aq.data_ptr(), aq.stride(0), a_s.data_ptr(), a_s.stride(0), M,
                               bq.data_ptr(), bq.stride(0), b_s.data_ptr(), b_s.stride(0), N, Kdim,
                               out.data_ptr(), ldc, dt, ws.data_ptr(), ws.numel(), _stream(stream))
    _check(st, "fp4q_mxfp8_gemm")
    return out


def _out_buffer(rows: int, cols: int, dt: int, device):
    per16 = 8 if dt == OUT_BF16 else 4
    ld = max((cols + per16 - 1) // per16 * per16, per16)
    return torch.empty((rows, ld), dtype=_out_dtype(dt), device=device)[:, :cols]


def fp4q_gemm_fwd_act1d(xq, xs, T: int, W: QTensor, out=None, dt: int = OUT_BF16, ws=None, stream=None):
    """Y[T,N] = X^ W^^T with X in 1D blocks along the contraction axis (fp4q_quantize1d) and W in 2D blocks."""
    dev = xq.device
    if out is None:
        out = _out_buffer(T, W.rows, dt, dev)
    if ws is None:
        ws = alloc_workspace(dev)
    cw = W.c_struct()
    st = lib().fp4q_gemm_fwd_act1d(xq.data_ptr(), xq.stride(0), xs.data_ptr(), xs.stride(0), T, ctypes.byref(cw),
                                   out.data_ptr(), out.stride(0), dt, ws.data_ptr(), ws.numel(), _stream(stream))
    _check(st, "fp4q_gemm_fwd_act1d")
    return out


def fp4q_gemm_wgrad_act1d(dY: QTensor, xtq, xts, K: int, out=None, dt: int = OUT_F32, accumulate: bool = False,
                          ws=None, stream=None):
    """dW[N,K] (+)= dY^^T X^_t with X^_t the 1D-block encoding of X^T (fp4q_quantize1d_t) and dY in 2D blocks."""
    dev = xtq.device
    if out is None:
        out = _out_buffer(dY.cols, K, dt, dev)
        if accumulate:
            out.zero_()
    if ws is None:
        ws = alloc_workspace(dev)
    cd = dY.c_struct()
    st = lib().fp4q_gemm_wgrad_act1d(ctypes.byref(cd), xtq.data_ptr(), xtq.stride(0), xts.data_ptr(), xts.stride(0), K,
                                     out.data_ptr(), out.stride(0), dt, 1 if accumulate else 0, ws.data_ptr(),
                                     ws.numel(), _stream(stream))
    _check(st, "fp4q_gemm_wgrad_act1d")
    return out


def fp4q_workspace_bytes() -> int:
    return int(lib().fp4q_workspace_bytes())


def alloc_workspace(device) -> torch.Tensor:
    return torch.zeros(fp4q_workspace_bytes(), dtype=torch.uint8, device=device)


def fp4q_workspace_status(ws: torch.Tensor, stream=None) -> int:
    return int(lib().fp4q_workspace_status(ws.data_ptr(), _stream(stream)))


def fp4q_workspace_set_wait_limit(ws: torch.Tensor, polls: int, stream=None):
    """Poll limit of the kernels' bounded waits for every later call that uses ws (0 = default)."""
    _check(lib().fp4q_workspace_set_wait_limit(ws.data_ptr(), int(polls), _stream(stream)), "fp4q_workspace_set_wait_limit")


def fp4q_debug_withhold_load(ws: torch.Tensor, nth_load: int, stream=None):
    """Development aid: the first CTA of later GEMM calls on ws leaves out its n-th operand load (0 = off)."""
    _check(lib().fp4q_debug_withhold_load(ws.data_ptr(), int(nth_load), _stream(stream)), "fp4q_debug_withhold_load")


def _groups(row_offsets: Optional[torch.Tensor], row_alignment: int = 128):
    if row_offsets is None:
        return None, None
    _dev(row_offsets, "row_offsets")
    if row_offsets.dtype != torch.int64 or not row_offsets.is_contiguous():
        raise ValueError("row_offsets must be a contiguous int64 device tensor")
    g = _CGroups(row_offsets.numel() - 1, row_alignment, row_offsets.data_ptr())
    return g, ctypes.byref(g)


def _out_dtype(dt: int):
    return torch.bfloat16 if dt == OUT_BF16 else torch.float32


def _gemm(fn_name, a: QTensor, b: QTensor, out_rows, out_cols, out, dt, row_offsets, ws, stream, accumulate=None,
          row_alignment: int = 128):
    dev = a.q_rm.device
    if out is None:
        # the ABI wants the leading dimension to be a multiple of 16 bytes: pad it and return a view
        per16 = 8 if dt == OUT_BF16 else 4
        ld = max((out_cols + per16 - 1) // per16 * per16, per16)
        out = torch.empty((out_rows, ld), dtype=_out_dtype(dt), device=dev)[:, :out_cols]
    if ws is None:
        ws = alloc_workspace(dev)
    ca, cb = a.c_struct(), b.c_struct()
    g, gref = _groups(row_offsets, row_alignment)
    fn = getattr(lib(), fn_name)
    args = [ctypes.byref(ca), ctypes.byref(cb), out.data_ptr(), out.stride(0) if out.numel() else out_cols, dt]
    if accumulate is not None:
        args.append(int(accumulate))
    args += [gref, ws.data_ptr(), ws.numel(), _stream(stream)]
    _check(fn(*args), fn_name)
    return out


def fp4q_gemm_fwd(X: QTensor, W: QTensor, out=None, dt: int = OUT_BF16, row_offsets=None, ws=None, stream=None,
                  row_alignment: int = 128):
    """Y[T,N] = X^ W^^T. Grouped when row_offsets is given (W is then the expert stack [E*N, K])."""
    n = W.rows if row_offsets is None else W.rows // (row_offsets.numel() - 1)
    return _gemm("fp4q_gemm_fwd", X, W, X.rows, n, out, dt, row_offsets, ws, stream, row_alignment=row_alignment)


def fp4q_gemm_fwd_quantized(X: QTensor, W: QTensor, out: Optional[QTensor] = None, mode: int = ROUND_NEAREST,
                            seed: int = 0, tensor_id: int = 0, want_t: bool = True, ws=None, stream=None,
                            row_offsets=None) -> QTensor:
    """Yq = 2D-block FP4 of the BF16-rounded product X^ W^^T, quantized in the GEMM's epilogue.  Grouped when
    row_offsets is given (every group then starts on a multiple of 256 rows)."""
    dev = X.q_rm.device
    g, gref = _groups(row_offsets, 256)
    if out is None:
        out = alloc_qtensor(X.rows, W.rows if row_offsets is None else W.rows // (row_offsets.numel() - 1), dev, want_t)
    if ws is None:
        ws = alloc_workspace(dev)
    cx, cw, cy = X.c_struct(), W.c_struct(), out.c_struct()
    st = lib().fp4q_gemm_fwd_quantized(ctypes.byref(cx), ctypes.byref(cw), ctypes.byref(cy), mode, seed, tensor_id, gref,
                                       ws.data_ptr(), ws.numel(), _stream(stream))
    _check(st, "fp4q_gemm_fwd_quantized")
    return out


def fp4q_gemm_dgrad_quantized(dY: QTensor, W: QTensor, out: Optional[QTensor] = None, mode: int = ROUND_STOCHASTIC,
                              seed: int = 0, tensor_id: int = 0, want_t: bool = True, ws=None, stream=None,
                              row_offsets=None) -> QTensor:
    """dXq = 2D-block FP4 of the BF16-rounded product dY^ W^, quantized in the GEMM's epilogue.  Grouped when
    row_offsets is given (every group then starts on a multiple of 256 rows)."""
    dev = dY.q_rm.device
    g, gref = _groups(row_offsets, 256)
    if out is None:
        out = alloc_qtensor(dY.rows, W.cols, dev, want_t)
    if ws is None:
        ws = alloc_workspace(dev)
    cd, cw, cx = dY.c_struct(), W.c_struct(), out.c_struct()
    st = lib().fp4q_gemm_dgrad_quantized(ctypes.byref(cd), ctypes.byref(cw), ctypes.byref(cx), mode, seed, tensor_id, gref,
                                         ws.data_ptr(), ws.numel(), _stream(stream))
    _check(st, "fp4q_gemm_dgrad_quantized")
    return out


def fp4q_gemm_fwd_static_workspace(X: QTensor, W: QTensor, out: torch.Tensor, dt: int = OUT_BF16,
                                   status_out: Optional[torch.Tensor] = None, stream=None):
    """Y = X^ W^^T through the entry point that allocates nothing: the caller supplies the output (and,
    optionally, a 4-byte device tensor for the kernel's status word); the workspace is the library's own
    fixed array.  Nothing is allocated here either."""
    cx, cw = X.c_struct(), W.c_struct()
    st = lib().fp4q_gemm_fwd_static_workspace(ctypes.byref(cx), ctypes.byref(cw), out.data_ptr(), out.stride(0), dt,
                                              status_out.data_ptr() if status_out is not None else None,
                                              _stream(stream))
    _check(st, "fp4q_gemm_fwd_static_workspace")
    return out


def fp4q_gemm_dgrad(dY: QTensor, W: QTensor, out=None, dt: int = OUT_BF16, row_offsets=None, ws=None, stream=None,
                    row_alignment: int = 128):
    """dX[T,K] = dY^ W^."""
    return _gemm("fp4q_gemm_dgrad", dY, W, dY.rows, W.cols, out, dt, row_offsets, ws, stream, row_alignment=row_alignment)


def fp4q_gemm_wgrad(dY: QTensor, X: QTensor, out=None, dt: int = OUT_F32, accumulate: bool = False,
                    row_offsets=None, ws=None, stream=None):
    """dW[N,K] = dY^^T X^ (stack [E*N, K] when grouped)."""
    e = 1 if row_offsets is None else row_offsets.numel() - 1
    return _gemm("fp4q_gemm_wgrad", dY, X, dY.cols * e, X.cols, out, dt, row_offsets, ws, stream,
                 accumulate=accumulate)


def _gemm_b16(fn_name, a: QTensor, b: QTensor, out_rows, out_cols, out, dt, ws, stream, accumulate=None):
    dev = a.q_rm.device
    if out is None:
        out = _out_buffer(out_rows, out_cols, dt, dev)
        if accumulate:
            out.zero_()
    if ws is None:
        ws = alloc_workspace(dev)
    ca, cb = a.c_struct(16), b.c_struct(16)
    args = [ctypes.byref(ca), ctypes.byref(cb), out.data_ptr(), out.stride(0) if out.numel() else out_cols, dt]
    if accumulate is not None:
        args.append(int(accumulate))
    args += [ws.data_ptr(), ws.numel(), _stream(stream)]
    _check(getattr(lib(), fn_name)(*args), fn_name)
    return out


def fp4q_gemm_fwd_b16(X: QTensor, W: QTensor, out=None, dt: int = OUT_BF16, ws=None, stream=None):
    """Y[T,N] = X^ W^^T on tensors quantized in 16 x 16 blocks (fp4q_quantize2d with BLOCK_16)."""
    return _gemm_b16("fp4q_gemm_fwd_b16", X, W, X.rows, W.rows, out, dt, ws, stream)


def fp4q_gemm_dgrad_b16(dY: QTensor, W: QTensor, out=None, dt: int = OUT_BF16, ws=None, stream=None):
    """dX[T,K] = dY^ W^ on tensors quantized in 16 x 16 blocks."""
    return _gemm_b16("fp4q_gemm_dgrad_b16", dY, W, dY.rows, W.cols, out, dt, ws, stream)


def fp4q_gemm_wgrad_b16(dY: QTensor, X: QTensor, out=None, dt: int = OUT_F32, accumulate: bool = False, ws=None, stream=None):
    """dW[N,K] (+)= dY^^T X^ on tensors quantized in 16 x 16 blocks."""
    return _gemm_b16("fp4q_gemm_wgrad_b16", dY, X, dY.cols, X.cols, out, dt, ws, stream, accumulate=accumulate)


def fp4q_mxfp8_qk(xq, xs, wq_q, wq_s, wk_q, wk_s, T: int, K: int, N: int, dt: int = OUT_BF16, ws=None,
                  stream=None):
    """Q = X^ Wq^^T and K = X^ Wk^^T on MXFP8 operands from fp4q_mxfp8_quantize1d."""
    dev = xq.device
    per16 = 8 if dt == OUT_BF16 else 4
    ldo = max((N + per16 - 1) // per16 * per16, per16)
    q_out = torch.empty((T, ldo), dtype=_out_dtype(dt), device=dev)[:, :N] if wq_q is not None else None
    k_out = torch.empty((T, ldo), dtype=_out_dtype(dt), device=dev)[:, :N] if wk_q is not None else None
    if ws is None:
        ws = alloc_workspace(dev)
    wref = wq_q if wq_q is not None else wk_q
    sref = wq_s if wq_s is not None else wk_s
    p = lambda t: t.data_ptr() if t is not None else None
    st = lib().fp4q_mxfp8_qk(xq.data_ptr(), xq.stride(0), xs.data_ptr(), xs.stride(0), T, K,
                             p(wq_q), p(wq_s), p(wk_q), p(wk_s), wref.stride(0), sref.stride(0), N,
                             p(q_out), p(k_out), ldo, dt, ws.data_ptr(), ws.numel(), _stream(stream))
    _check(st, "fp4q_mxfp8_qk")
    return q_out, k_out
