"""GPU parity of the block-size variants of the 2D quantizer (block-size study, Table 4 of the paper): 16 x 16 and
64 x 64 blocks against the oracle's free-block-size quantizer, bit for bit; 64-block and 16-block tensors as GEMM
operands (the latter through the products on 16-element scale vectors) against the oracle's products."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import bits_tensor, check_gemm

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


def _deq16(x, qt):
    """Oracle dequantization of the GPU's own 16-block payload (checked bit-exact by `check` before)."""
    rows, cols = x.shape
    o = oracle.quantize2d_block(workloads.bf16_bits(x), 16, want_t=False)
    return oracle.dequantize2d_block(o[0], o[2], 16, rows, cols)


def _three_products_b16(x, w, dy, dt=binding.OUT_F32, mode=binding.ROUND_NEAREST):
    X, W, dY = check(x, 16, mode), check(w, 16, mode), check(dy, 16, mode)
    ws = binding.alloc_workspace("cuda")
    y = binding.fp4q_gemm_fwd_b16(X, W, dt=dt, ws=ws)
    dx = binding.fp4q_gemm_dgrad_b16(dY, W, dt=dt, ws=ws)
    dw = binding.fp4q_gemm_wgrad_b16(dY, X, dt=binding.OUT_F32, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    xd, wd, dyd = _deq16(x, X), _deq16(w, W), _deq16(dy, dY)
    return (y, oracle.gemm_fwd(xd, wd)), (dx, oracle.gemm_dgrad(dyd, wd)), (dw, oracle.gemm_wgrad(dyd, xd))


@pytest.mark.parametrize("T,N,K", [(128, 256, 256), (256, 512, 512), (384, 640, 1024), (200, 136, 416), (1000, 1152, 2304)])
def test_a_16_block_tensor_feeds_the_gemm(T, N, K):
    x = workloads.activations_gauss_outliers(T, K, seed=8, device="cuda")
    w = workloads.weights(N, K, seed=9, device="cuda")
    dy = workloads.gradients_rowscaled(T, N, seed=10, device="cuda")
    for (got, ref), name in zip(_three_products_b16(x, w, dy, dt=binding.OUT_BF16 if T & 8 else binding.OUT_F32), ("fwd", "dgrad", "wgrad")):
        check_gemm(got, ref, "%s on 16-block tensors %dx%dx%d" % (name, T, N, K))


def test_16_block_products_scale_layout_probe_and_exact_case():
    # every 16 x 16 block gets its own power-of-two magnitude: a scale byte read for the wrong 16 rows or the wrong 16
    # contraction elements changes the result by a factor >= 2
    g = torch.Generator(device="cuda").manual_seed(3)

    def spread(r, c, a, b, m):
        i = torch.arange(r, device="cuda")[:, None] // 16
        j = torch.arange(c, device="cuda")[None, :] // 16
        return (torch.randn(r, c, generator=g, device="cuda") * torch.exp2(((a * i + b * j) % m).float() - m // 2)).to(torch.bfloat16)

    for (got, ref), name in zip(_three_products_b16(spread(384, 640, 1, 2, 11), spread(512, 640, 3, 1, 13), spread(384, 512, 2, 3, 7)),
                                ("fwd", "dgrad", "wgrad")):
        check_gemm(got, ref, name + ", distinct scale per 16 x 16 block")
    # operands on the E2M1 grid times a power of two per block: every partial sum is exact in FP32 -> bit for bit
    grid = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6], device="cuda")

    def draw(r, c, e0):
        v = grid[torch.randint(0, 8, (r, c), generator=g, device="cuda")]
        sgn = torch.randint(0, 2, (r, c), generator=g, device="cuda") * 2 - 1
        i = torch.arange(r, device="cuda")[:, None] // 16
        j = torch.arange(c, device="cuda")[None, :] // 16
        return (v * sgn * torch.exp2(((i + j) % 3 + e0).float())).to(torch.bfloat16)

    for (got, ref), name in zip(_three_products_b16(draw(256, 512, -3), draw(384, 512, 2), draw(256, 384, -1)), ("fwd", "dgrad", "wgrad")):
        assert np.array_equal(got.double().cpu().numpy(), ref), name + ": exact case differs"


def test_block_sizes_must_match_the_product():
    x = workloads.weights(64, 64, 1, "cuda")
    X = binding.fp4q_quantize2d(x, flags=binding.BLOCK_16)
    with pytest.raises(ValueError):
        binding.fp4q_gemm_fwd(X, X)                                  # the 32-block products refuse a 16-block tensor
    with pytest.raises(ValueError):
        binding.fp4q_gemm_fwd_b16(binding.fp4q_quantize2d(x), X)      # and the 16-block products a 32-block one
    with pytest.raises(binding.Fp4qError):
        binding.fp4q_quantize2d(x, flags=binding.BLOCK_16 | binding.BLOCK_64)
