import ctypes
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def library_pins():
    """Host-side wrappers around library routines (cuda_fp4.h, cuda_fp8.h, cuRAND and ATen Philox)
    that pin the oracle from outside. Built on demand with nvcc (host code only); tests that need it
    are skipped if the toolchain cannot build it."""
    here = os.path.join(ROOT, "tests", "helpers")
    src = os.path.join(here, "library_pins.cu")
    so = os.path.join(here, "liblibrary_pins.so")
    if not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
        try:
            import torch
            inc = os.path.join(os.path.dirname(torch.__file__), "include")
            tmp = so + ".%d.tmp" % os.getpid()
            subprocess.run(["nvcc", "-O1", "-shared", "-Xcompiler", "-fPIC", "-std=c++17",
                            "-Wno-deprecated-gpu-targets", "--expt-relaxed-constexpr", "-I" + inc,
                            "-o", tmp, src], check=True, capture_output=True)
            os.replace(tmp, so)
        except Exception as exc:  # pragma: no cover - toolchain missing
            pytest.skip("cannot build library pins: %r" % (exc,))
    L = ctypes.CDLL(so)
    L.pin_fp4_decode.restype = ctypes.c_float
    L.pin_fp4_decode.argtypes = [ctypes.c_int]
    L.pin_fp4_encode_rn.restype = ctypes.c_int
    L.pin_fp4_encode_rn.argtypes = [ctypes.c_float]
    L.pin_e4m3_encode_rn.restype = ctypes.c_int
    L.pin_e4m3_encode_rn.argtypes = [ctypes.c_float]
    L.pin_e4m3_decode.restype = ctypes.c_float
    L.pin_e4m3_decode.argtypes = [ctypes.c_int]
    L.pin_e8m0_encode_ceil.restype = ctypes.c_int
    L.pin_e8m0_encode_ceil.argtypes = [ctypes.c_float]
    L.pin_philox_curand.restype = None
    L.pin_philox_curand.argtypes = [ctypes.c_void_p] * 3
    L.pin_philox_aten.restype = None
    L.pin_philox_aten.argtypes = [ctypes.c_uint64] * 3 + [ctypes.c_void_p]
    return L
