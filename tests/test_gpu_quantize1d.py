"""GPU parity: the 1D-block (1 x 32) FP4 quantizers of activations (Section 3.1 keeps this layout for activations)
against the CPU oracle, bit for bit, through the C ABI - blocks along the rows (forward operand) and the encoding
of the transpose (weight-gradient operand) - and the Figure 1 transposition diagnostic computed from GPU outputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import bits_tensor

pytestmark = pytest.mark.gpu

MODES = [binding.ROUND_NEAREST, binding.ROUND_STOCHASTIC]


def check_rowwise(x, mode=binding.ROUND_NEAREST, seed=0, tensor_id=0):
    rows, cols = x.shape
    q, s = binding.fp4q_quantize1d(x, mode, seed, tensor_id)
    torch.cuda.synchronize()
    oq, os_ = oracle.quantize1d(workloads.bf16_bits(x), mode, seed, tensor_id)
    gq, gs = q.cpu().numpy(), s.cpu().numpy()
    assert np.array_equal(gs[:, :os_.shape[1]], os_), "scales differ"
    assert np.array_equal(gq[:, :oq.shape[1]], oq), "payload differs"
    assert not gq[:, oq.shape[1]:(cols + 31) // 32 * 16].any(), "block padding is not zero"
    return gq, gs


def check_transposed(x):
    rows, cols = x.shape
    q, s = binding.fp4q_quantize1d_t(x)
    torch.cuda.synchronize()
    oq, os_ = oracle.quantize1d_t(workloads.bf16_bits(x))
    gq, gs = q.cpu().numpy(), s.cpu().numpy()
    assert np.array_equal(gs[:, :os_.shape[1]], os_), "scales differ"
    assert np.array_equal(gq[:, :oq.shape[1]], oq), "payload differs"
    assert not gq[:, oq.shape[1]:(rows + 31) // 32 * 16].any(), "block padding is not zero"
    return gq, gs


def _random_finite_bits(rng, rows, cols):
    b = rng.integers(0, 1 << 16, size=(rows, cols), dtype=np.uint32).astype(np.uint16)
    nonfinite = (b & 0x7F80) == 0x7F80
    b[nonfinite] &= 0xBFFF
    return b


@pytest.mark.parametrize("mode", MODES)
def test_activations_rowwise(mode):
    x = workloads.activations_gauss_outliers(384, 512, seed=3, device="cuda")
    check_rowwise(x, mode, seed=5, tensor_id=1)
    x = workloads.activations_student_t(160, 1024, seed=4, device="cuda")
    check_rowwise(x, mode, seed=6, tensor_id=2)


@pytest.mark.parametrize("mode", MODES)
def test_random_bit_patterns_rowwise(mode):
    rng = np.random.default_rng(1)
    check_rowwise(bits_tensor(_random_finite_bits(rng, 96, 416)), mode, seed=9, tensor_id=3)


def test_ragged_shapes_rowwise():
    rng = np.random.default_rng(2)
    for rows, cols in [(1, 1), (3, 31), (5, 33), (7, 100), (33, 250), (2, 48)]:
        check_rowwise(bits_tensor(_random_finite_bits(rng, rows, cols)))
    # stochastic rounding with a 16-element ragged tail
    check_rowwise(bits_tensor(_random_finite_bits(rng, 9, 80)), binding.ROUND_STOCHASTIC, seed=1, tensor_id=7)


def test_nonfinite_and_zero_blocks_rowwise():
    rng = np.random.default_rng(3)
    b = _random_finite_bits(rng, 16, 128)
    b[0, 3] = 0x7F80      # +Inf
    b[1, 40] = 0xFF80     # -Inf
    b[2, 70] = 0x7FC1     # NaN
    b[3, :32] = 0         # all-zero block
    b[4, 32:64] = 0x8000  # all negative zero
    b[5, 64:96] = 0x7F80  # a block with no finite element
    for mode in MODES:
        check_rowwise(bits_tensor(b), mode, seed=2, tensor_id=4)


def test_activations_transposed():
    x = workloads.activations_gauss_outliers(384, 512, seed=3, device="cuda")
    check_transposed(x)
    x = workloads.activations_student_t(1024, 192, seed=4, device="cuda")
    check_transposed(x)
    rng = np.random.default_rng(4)
    check_transposed(bits_tensor(_random_finite_bits(rng, 160, 320)))


def test_ragged_and_nonfinite_transposed():
    rng = np.random.default_rng(5)
    for rows, cols in [(1, 1), (31, 3), (33, 5), (100, 7), (250, 65), (64, 63), (129, 130)]:
        check_transposed(bits_tensor(_random_finite_bits(rng, rows, cols)))
    b = _random_finite_bits(rng, 96, 64)
    b[3, 0] = 0x7F80
    b[40, 1] = 0xFF80
    b[70, 2] = 0x7FC1
    b[:32, 3] = 0
    b[32:64, 4] = 0x7F80
    check_transposed(bits_tensor(b))


def test_transposed_tile_path_with_nonfinite_values_and_all_scale_codes():
    # shapes made of full 128 x 128 tiles take the tile kernel: random bit patterns (every exponent), zero column
    # blocks, +-Inf, NaN, a column block without a finite entry
    rng = np.random.default_rng(6)
    b = _random_finite_bits(rng, 256, 384)
    check_transposed(bits_tensor(b))
    b[3, 5] = 0x7F80
    b[40, 70] = 0xFF80
    b[100, 200] = 0x7FC1
    b[128:160, 17] = 0
    b[160:192, 18] = 0x8000
    b[192:224, 19] = 0x7F80
    check_transposed(bits_tensor(b))
    check_transposed(workloads.activations_gauss_outliers(512, 256, seed=9, device="cuda"))


def test_empty_and_rejected_arguments():
    e = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    q, s = binding.fp4q_quantize1d(e)
    assert q.shape[0] == 0
    q, s = binding.fp4q_quantize1d_t(e)
    assert q.shape[0] == 64
    x = torch.zeros((4, 40), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.Fp4qError):
        binding.fp4q_quantize1d(x, binding.ROUND_STOCHASTIC)   # stochastic rounding wants cols % 16 == 0


def test_transposition_diagnostic_from_gpu_encodings():
    """Figure 1 (c), (d): with 1D blocks an element's scale exponent depends on the orientation it is quantized in;
    with 2D blocks it does not.  The maps are formed from the GPU quantizers' scales and agree with the oracle's."""
    x = workloads.activations_gauss_outliers(256, 256, seed=8, device="cuda")
    _, s_fwd = binding.fp4q_quantize1d(x)
    _, s_bwd = binding.fp4q_quantize1d_t(x)
    torch.cuda.synchronize()
    e_fwd = np.repeat(s_fwd.cpu().numpy().astype(np.int32), 32, axis=1)
    e_bwd = np.repeat(s_bwd.cpu().numpy().astype(np.int32), 32, axis=1).T
    d1 = e_fwd - e_bwd
    ref = oracle.transposition_diagnostic(workloads.bf16_bits(x))
    assert np.array_equal(d1, ref["scale_exponent_difference_1d"])
    assert np.abs(d1).mean() > 0.5
