"""GPU parity of the MXFP8 backward path (Section 3.2 applies MXFP8 to the query/key projections; the backward
products re-quantize their operands along the new contraction axis): the transposing quantizer bit for bit against
the oracle, and dX = dY W, dW = dY^T X against the oracle's products within the GEMM tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def check(got, ref, what):
    g = got.double().cpu().numpy()
    if got.dtype == torch.bfloat16:
        ref = oracle.bf16_round(ref)
    rel = np.linalg.norm(g - ref) / np.linalg.norm(ref)
    assert rel <= 1e-3, "%s: relative Frobenius error %.3e" % (what, rel)
    row_inf = np.abs(ref).max(axis=1, keepdims=True)
    assert (np.abs(g - ref) <= 1e-2 * row_inf + 1e-300).all(), "%s: per-row max-abs bound violated" % what


def quantize_t_checked(x):
    """Transposed MXFP8 operand from the GPU, checked bit for bit against the oracle; returns (q, s, dequantized)."""
    rows, cols = x.shape
    q, s = binding.fp4q_mxfp8_quantize1d_t(x)
    torch.cuda.synchronize()
    oq, os_ = oracle.mxfp8_quantize1d_t(workloads.bf16_bits(x))
    assert np.array_equal(s.cpu().numpy()[:, :(rows + 31) // 32], os_), "scales differ"
    gq = q.cpu().numpy()
    assert np.array_equal(gq[:, :rows], oq), "payload differs"
    assert not gq[:, rows:(rows + 31) // 32 * 32].any(), "block padding is not zero"
    return q, s, oracle.mxfp8_dequantize(oq, os_)


def quantize_checked(x):
    rows, cols = x.shape
    q, s = binding.fp4q_mxfp8_quantize1d(x)
    torch.cuda.synchronize()
    oq, os_ = oracle.mxfp8_quantize1d(workloads.bf16_bits(x))
    assert np.array_equal(s.cpu().numpy()[:, :(cols + 31) // 32], os_)
    assert np.array_equal(q.cpu().numpy()[:, :cols], oq)
    return q, s, oracle.mxfp8_dequantize(oq, os_)


@pytest.mark.parametrize("rows,cols", [(32, 64), (100, 70), (257, 129), (1, 1), (512, 1000), (65, 2)])
def test_transposing_quantizer_matches_the_oracle(rows, cols):
    x = workloads.activations_student_t(rows, cols, 900 + rows, "cuda")
    quantize_t_checked(x)


def test_transposing_quantizer_edge_values():
    bits = np.zeros((96, 4), dtype=np.uint16)
    bits[:32, 0] = 0x43E0                      # 448 everywhere: scale 1
    bits[32, 0] = 0x43E1                       # just above 448 in the next block: scale 2
    bits[:, 1] = np.arange(96) | 0x3F00
    bits[5, 2], bits[6, 2], bits[7, 2] = 0x7F80, 0xFF80, 0x7FC0    # +Inf, -Inf, NaN
    bits[:64, 3] = np.arange(64)               # subnormals
    quantize_t_checked(workloads.bits_to_bf16(bits, "cuda"))


@pytest.mark.parametrize("T,N,K", [(128, 256, 256), (200, 136, 416), (1024, 512, 768)])
def test_backward_products_of_an_mxfp8_projection(T, N, K):
    X = workloads.activations_student_t(T, K, 910, "cuda")
    W = workloads.weights(N, K, 911, "cuda")
    dY = workloads.gradients_rowscaled(T, N, 912, "cuda")
    ws = binding.alloc_workspace("cuda")
    dyq, dys, dyd = quantize_checked(dY)            # [T, N], blocks along N
    wtq, wts, wtd = quantize_t_checked(W)           # [K, N], blocks along N
    dx = binding.fp4q_mxfp8_gemm(dyq, dys, wtq, wts, T, K, N, dt=binding.OUT_BF16, ws=ws)
    dytq, dyts, dytd = quantize_t_checked(dY)       # [N, T], blocks along T
    xtq, xts, xtd = quantize_t_checked(X)           # [K, T], blocks along T
    dw = binding.fp4q_mxfp8_gemm(dytq, dyts, xtq, xts, N, K, T, dt=binding.OUT_F32, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    check(dx, dyd @ wtd.T, "dgrad")                 # dX[t,k] = sum_n dY^[t,n] W^T^[k,n]
    check(dw, dytd @ xtd.T, "wgrad")                # dW[n,k] = sum_t dY^T^[n,t] X^T^[k,t]


def test_transposing_quantizer_tile_path_with_nonfinite_values():
    # shapes made of full 128 x 128 tiles take the tile kernel: random bit patterns (every exponent), zero column
    # blocks, +-Inf, NaN, a column block without a finite entry
    rng = np.random.default_rng(16)
    b = rng.integers(0, 1 << 16, size=(256, 384), dtype=np.uint32).astype(np.uint16)
    b[(b & 0x7F80) == 0x7F80] &= 0xBFFF
    quantize_t_checked(workloads.bits_to_bf16(b, "cuda"))
    b[3, 5] = 0x7F80
    b[40, 70] = 0xFF80
    b[100, 200] = 0x7FC1
    b[128:160, 17] = 0
    b[160:192, 18] = 0x8000
    b[192:224, 19] = 0x7F80
    quantize_t_checked(workloads.bits_to_bf16(b, "cuda"))
    quantize_t_checked(workloads.activations_gauss_outliers(512, 256, seed=9, device="cuda"))
