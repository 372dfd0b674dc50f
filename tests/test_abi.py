"""CPU-side checks of the C boundary: the library loads, exports every symbol the header declares, and
rejects bad arguments before touching the GPU (no compute calls here)."""
import ctypes
import os
import re

import pytest

from paper_2607_24953_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fp4q.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fp4q_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = binding.lib()
    names = declared_functions()
    assert {"fp4q_quantize2d", "fp4q_gemm_fwd", "fp4q_gemm_dgrad", "fp4q_gemm_wgrad", "fp4q_mxfp8_qk"} <= set(names)
    for n in names:
        assert hasattr(L, n), "libfp4q.so does not export %s" % n
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings_and_version():
    assert binding.status_string(0) == "ok"
    assert "NULL" in binding.status_string(1)
    assert binding.lib().fp4q_version() >= 100
    assert binding.fp4q_workspace_bytes() >= 8


def _tensor(rows, cols, q_rm=16, ld_rm=None, q_t=32, ld_t=None, scale=48, ld_s=None):
    return binding._CTensor(rows, cols, q_rm, ld_rm if ld_rm is not None else (cols + 31) // 32 * 16,
                            q_t, ld_t if ld_t is not None else (rows + 31) // 32 * 16,
                            scale, ld_s if ld_s is not None else (cols + 31) // 32)


def test_quantize2d_argument_validation():
    L = binding.lib()
    q = lambda x, r, c, ld, t, mode=0, flags=0: L.fp4q_quantize2d(x, r, c, ld, ctypes.byref(t) if t else None, mode, 0, 0, flags, None)
    t = _tensor(64, 64)
    assert q(0x1000, -1, 64, 64, t) == 2                      # negative size
    assert q(0x1000, 64, 64, 64, None) == 1                   # NULL descriptor
    assert q(None, 64, 64, 64, t) == 1                        # NULL input
    assert q(0x1000, 64, 64, 32, t) == 2                      # ld_x < cols
    assert q(0x1000, 64, 64, 64, _tensor(64, 32)) == 2        # descriptor shape mismatch
    assert q(0x1000, 64, 64, 64, _tensor(64, 64, ld_rm=16)) == 2   # payload pitch too small
    assert q(0x1000, 64, 64, 64, _tensor(64, 64, ld_rm=40)) == 3   # pitch not a multiple of 16
    assert q(0x1000, 64, 64, 64, _tensor(64, 64, q_rm=8)) == 3     # misaligned payload
    assert q(0x1001, 64, 64, 64, t) == 3                      # odd input address
    assert q(0x1000, 64, 64, 64, t, mode=2) == 4              # unknown rounding mode
    assert q(0x1000, 64, 64, 64, t, flags=8) == 4             # unknown flag
    assert q(None, 0, 64, 64, _tensor(0, 64)) == 0            # empty input is a no-op


def test_gemm_argument_validation():
    L = binding.lib()
    X, W = _tensor(128, 256), _tensor(64, 256)
    bad_w = _tensor(64, 128)
    call = lambda x, w, y, ldy, dt=0, ws=0x100, wsb=256: L.fp4q_gemm_fwd(ctypes.byref(x), ctypes.byref(w), y, ldy, dt, None, ws, wsb, None)
    assert call(X, bad_w, 0x1000, 64) == 2                    # contraction lengths differ
    assert call(X, W, None, 64) == 1                          # NULL output
    assert call(X, W, 0x1000, 32) == 2                        # ldy < N
    assert call(X, W, 0x1000, 64, dt=7) == 4
    assert call(X, W, 0x1000, 64, ws=None) == 5               # no workspace
    assert call(X, W, 0x1000, 64, wsb=4) == 5                 # workspace too small
    assert call(X, W, 0x1008, 64) == 3                        # misaligned output
    assert call(X, W, 0x1000, 68) == 3                        # output pitch not a multiple of 16 bytes
    assert call(_tensor(0, 256), W, None, 64) == 0            # no rows: no-op
    assert L.fp4q_gemm_wgrad(ctypes.byref(X), ctypes.byref(_tensor(128, 64)), 0x1000, 64, 0, 1, None, 0x100, 256, None) == 4  # accumulate needs FP32
    assert L.fp4q_gemm_dgrad(ctypes.byref(X), ctypes.byref(_tensor(100, 64)), 0x1000, 64, 0, None, 0x100, 256, None) == 2


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError):
        binding.fp4q_quantize2d(torch.zeros(32, 32, dtype=torch.bfloat16))
