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
