"""GPU parity of the block-size variants of the 2D quantizer (block-size study, Table 4 of the paper): 16 x 16 and
64 x 64 blocks against the oracle's free-block-size quantizer, bit for bit; a 64-block tensor as a GEMM operand."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import bits_tensor

pytestmark = pytest.mark.gpu

FLAG = {16: binding.BLOCK_16, 64: binding.BLOCK_64}


def check(x, b, mode, seed=0, tensor_id=0):
    rows, cols = x.shape
    qt = binding.fp4q_quantize2d(x, mode=mode, seed=seed, tensor_id=tensor_id, flags=FLAG[b])
    torch.cuda.synchronize()
    o_rm, o_t, o_s = oracle.quantize2d_block(workloads.bf16_bits(x), b, mode, seed, tensor_id)
    g_rm, g_t, g_s = qt.q_rm.cpu().numpy(), qt.q_t.cpu().numpy(), qt.scale.cpu().numpy()
    if b == 64:   # the library writes each block's scale to its four 32-granular entries
        o_s = np.repeat(np.repeat(o_s, 2, 0), 2, 1)[:(rows + 31) // 32, :(cols + 31) // 32]
    assert np.array_equal(g_s[:, :o_s.shape[1]], o_s), "scales differ"
    assert np.array_equal(g_rm[:, :o_rm.shape[1]], o_rm), "row-major payload differs"
    assert np.array_equal(g_t[:, :o_t.shape[1]], o_t), "transposed payload differs"
    return qt


def _random_finite_bits(rng, rows, cols):
    b = rng.integers(0, 1 << 16, size=(rows, cols), dtype=np.uint32).astype(np.uint16)
    b[(b & 0x7F80) == 0x7F80] &= 0xBFFF
    return b


@pytest.mark.parametrize("b", [16, 64])
@pytest.mark.parametrize("mode", [binding.ROUND_NEAREST, binding.ROUND_STOCHASTIC])
def test_workload_tensors(b, mode):
    check(workloads.activations_gauss_outliers(384, 512, seed=3, device="cuda"), b, mode, seed=5, tensor_id=1)
    check(workloads.gradients_rowscaled(256, 640, seed=4, device="cuda"), b, mode, seed=6, tensor_id=2)


@pytest.mark.parametrize("b", [16, 64])
@pytest.mark.parametrize("mode", [binding.ROUND_NEAREST, binding.ROUND_STOCHASTIC])
def test_random_bits_ragged_shapes_and_nonfinite_values(b, mode):
    rng = np.random.default_rng(b)
    for rows, cols in [(1, 1), (17, 33), (70, 65), (129, 200), (250, 48)]:
        check(bits_tensor(_random_finite_bits(rng, rows, cols)), b, mode, seed=9, tensor_id=3)
    bits = _random_finite_bits(rng, 128, 128)
    bits[3, 5] = 0x7F80        # +Inf
    bits[40, 70] = 0xFF80      # -Inf
    bits[100, 20] = 0x7FC1     # NaN
    bits[64:128, 64:128] = 0   # a zero 64-block
    bits[0:16, 112:128] = 0x7F80   # a 16-block without a finite entry
    check(bits_tensor(bits), b, mode, seed=2, tensor_id=4)


def test_a_64_block_tensor_feeds_the_gemm():
    T, N, K = 256, 256, 512
    x = workloads.activations_gauss_outliers(T, K, seed=8, device="cuda")
    w = workloads.weights(N, K, seed=9, device="cuda")
    X = check(x, 64, binding.ROUND_NEAREST)
    W = check(w, 64, binding.ROUND_NEAREST)
    y = binding.fp4q_gemm_fwd(X, W, dt=binding.OUT_F32)
    torch.cuda.synchronize()
    ox = oracle.quantize2d_block(workloads.bf16_bits(x), 64, want_t=False)
    ow = oracle.quantize2d_block(workloads.bf16_bits(w), 64, want_t=False)
    ref = oracle.gemm_fwd(oracle.dequantize2d_block(ox[0], ox[2], 64, T, K), oracle.dequantize2d_block(ow[0], ow[2], 64, N, K))
    g = y.double().cpu().numpy()
    assert np.linalg.norm(g - ref) / np.linalg.norm(ref) <= 1e-3
    assert (np.abs(g - ref) <= 1e-2 * np.abs(ref).max(axis=1, keepdims=True)).all()


def test_a_16_block_tensor_is_refused_as_a_gemm_operand():
    x = workloads.weights(64, 64, 1, "cuda")
    X = binding.fp4q_quantize2d(x, flags=binding.BLOCK_16)
    with pytest.raises(ValueError):
        binding.fp4q_gemm_fwd(X, X)
    with pytest.raises(binding.Fp4qError):
        binding.fp4q_quantize2d(x, flags=binding.BLOCK_16 | binding.BLOCK_64)
