"""GPU parity of fp4q_gemm_fwd_quantized: the forward product whose epilogue emits the 2D-block FP4 encoding of its
own BF16-rounded output.

Oracle: quantize2d(BF16(gemm_fwd(X^, W^))).  FP32 accumulation order is not the oracle's, so a bit-exact comparison
with the oracle needs operands for which every partial sum is exact (E2M1-grid values times a power of two): then
the GPU's BF16 output is the oracle's and payloads and scales must agree bit for bit.  On general operands the fused
call is compared, bit for bit, with the unfused chain (fp4q_gemm_fwd to BF16, then fp4q_quantize2d) and with the
oracle in two steps: the BF16 product against the oracle's product within the GEMM tolerance, and the fused payloads
and scales against the oracle's quantizer applied to that very BF16 product, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import assert_matches_oracle, check_gemm, dequant_from_gpu, logical

pytestmark = pytest.mark.gpu


def compare_logical(got, want_rm, want_t, want_s, rows, cols):
    g_rm, g_t, g_s = logical(got)
    assert np.array_equal(g_s, want_s), "scales differ"
    w = (cols + 1) // 2
    assert np.array_equal(g_rm[:, :w], want_rm[:, :w]), "row-major payload differs"
    assert not g_rm[:, w:(cols + 31) // 32 * 16].any(), "row-major block padding is not zero"
    h = (rows + 1) // 2
    assert np.array_equal(g_t[:, :h], want_t[:, :h]), "transposed payload differs"
    assert not g_t[:, h:(rows + 31) // 32 * 16].any(), "transposed block padding is not zero"


@pytest.mark.parametrize("T", [256, 200, 97])
@pytest.mark.parametrize("mode", [oracle.MODE_NEAREST, oracle.MODE_STOCHASTIC])
def test_exact_operands_match_the_oracle_bit_for_bit(T, mode):
    g = torch.Generator(device="cuda").manual_seed(5)
    grid = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6], device="cuda")

    def draw(r, c, e):
        v = grid[torch.randint(0, 8, (r, c), generator=g, device="cuda")]
        s = torch.randint(0, 2, (r, c), generator=g, device="cuda") * 2 - 1
        return (v * s * 2.0 ** e).to(torch.bfloat16)

    N, K = 400, 512
    X, W = draw(T, K, -3), draw(N, K, 5)
    qx = assert_matches_oracle(X, 0, seed=0, tensor_id=0)
    qw = assert_matches_oracle(W, 0, seed=0, tensor_id=1)
    xd, wd = dequant_from_gpu(qx), dequant_from_gpu(qw)
    ws = binding.alloc_workspace("cuda")
    yq = binding.fp4q_gemm_fwd_quantized(qx, qw, mode=mode, seed=9, tensor_id=4, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    y = oracle.bf16_round(oracle.gemm_fwd(xd, wd))                       # exact sums, rounded to BF16
    y_bits = workloads.bf16_bits(torch.from_numpy(y).to(torch.bfloat16))  # already representable: no second rounding
    o_rm, o_t, o_s = oracle.quantize2d(y_bits, mode, 9, 4)
    compare_logical(yq, o_rm, o_t, o_s, T, N)


@pytest.mark.parametrize("T,N,K", [(128, 256, 256), (300, 272, 1008), (1000, 1040, 320), (33, 16, 64)])
@pytest.mark.parametrize("mode", [0, 1])
def test_fused_equals_product_then_quantize(T, N, K, mode):
    X = workloads.activations_student_t(T, K, 700, "cuda")
    W = workloads.weights(N, K, 701, "cuda")
    qx = binding.fp4q_quantize2d(X, mode=0)
    qw = binding.fp4q_quantize2d(W, mode=0)
    ws = binding.alloc_workspace("cuda")
    fused = binding.fp4q_gemm_fwd_quantized(qx, qw, mode=mode, seed=3, tensor_id=8, ws=ws)
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_BF16, ws=ws)
    chain = binding.fp4q_quantize2d(y.contiguous(), mode=mode, seed=3, tensor_id=8)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    c_rm, c_t, c_s = logical(chain)
    compare_logical(fused, c_rm, c_t, c_s, T, N)


@pytest.mark.parametrize("T,N,K", [(300, 272, 1008), (1000, 1040, 320)])
@pytest.mark.parametrize("mode", [0, 1])
def test_general_operands_against_the_oracle_in_two_steps(T, N, K, mode):
    """General operands (FP32 accumulation order differs from the oracle's): the BF16 product is within the GEMM
    tolerance of the oracle's, and the fused encoding is exactly the oracle's quantizer applied to that BF16 product."""
    X = workloads.activations_student_t(T, K, 720, "cuda")
    W = workloads.weights(N, K, 721, "cuda")
    dY = workloads.gradients_rowscaled(T, N, 722, "cuda")
    qx = assert_matches_oracle(X, 0)
    qw = assert_matches_oracle(W, 0)
    qdy = assert_matches_oracle(dY, 1, seed=2, tensor_id=5)
    xd, wd, dyd = dequant_from_gpu(qx), dequant_from_gpu(qw), dequant_from_gpu(qdy)
    ws = binding.alloc_workspace("cuda")
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_BF16, ws=ws).contiguous()
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=binding.OUT_BF16, ws=ws).contiguous()
    fused_y = binding.fp4q_gemm_fwd_quantized(qx, qw, mode=mode, seed=3, tensor_id=8, ws=ws)
    fused_dx = binding.fp4q_gemm_dgrad_quantized(qdy, qw, mode=mode, seed=4, tensor_id=9, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    check_gemm(y, oracle.gemm_fwd(xd, wd), "forward product")
    check_gemm(dx, oracle.gemm_dgrad(dyd, wd), "input-gradient product")
    compare_logical(fused_y, *oracle.quantize2d(workloads.bf16_bits(y), mode, 3, 8), T, N)
    compare_logical(fused_dx, *oracle.quantize2d(workloads.bf16_bits(dx), mode, 4, 9), T, K)


def test_output_width_must_be_a_multiple_of_16():
    X = workloads.weights(64, 64, 1, "cuda")
    W = workloads.weights(40, 64, 2, "cuda")
    qx, qw = binding.fp4q_quantize2d(X), binding.fp4q_quantize2d(W)
    with pytest.raises(binding.Fp4qError):
        binding.fp4q_gemm_fwd_quantized(qx, qw)


@pytest.mark.parametrize("T,N,K", [(256, 256, 256), (300, 1000, 272), (1000, 320, 1040), (97, 64, 48)])
@pytest.mark.parametrize("mode", [0, 1])
def test_fused_dgrad_equals_product_then_quantize(T, N, K, mode):
    """dX = dY^ W^ quantized in the epilogue (the previous layer's dY) against fp4q_gemm_dgrad + fp4q_quantize2d."""
    dY = workloads.gradients_rowscaled(T, N, 710, "cuda")
    W = workloads.weights(N, K, 711, "cuda")
    qdy = binding.fp4q_quantize2d(dY, mode=1, seed=2, tensor_id=5)
    qw = binding.fp4q_quantize2d(W, mode=0)
    ws = binding.alloc_workspace("cuda")
    fused = binding.fp4q_gemm_dgrad_quantized(qdy, qw, mode=mode, seed=3, tensor_id=8, ws=ws)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=binding.OUT_BF16, ws=ws)
    chain = binding.fp4q_quantize2d(dx.contiguous(), mode=mode, seed=3, tensor_id=8)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    c_rm, c_t, c_s = logical(chain)
    compare_logical(fused, c_rm, c_t, c_s, T, K)


def test_fused_dgrad_exact_operands_match_the_oracle_bit_for_bit():
    g = torch.Generator(device="cuda").manual_seed(6)
    grid = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6], device="cuda")

    def draw(r, c, e):
        v = grid[torch.randint(0, 8, (r, c), generator=g, device="cuda")]
        s = torch.randint(0, 2, (r, c), generator=g, device="cuda") * 2 - 1
        return (v * s * 2.0 ** e).to(torch.bfloat16)

    T, N, K = 200, 512, 400
    dY, W = draw(T, N, -9), draw(N, K, 4)
    qdy = assert_matches_oracle(dY, 0, seed=0, tensor_id=0)
    qw = assert_matches_oracle(W, 0, seed=0, tensor_id=1)
    ws = binding.alloc_workspace("cuda")
    dxq = binding.fp4q_gemm_dgrad_quantized(qdy, qw, mode=oracle.MODE_STOCHASTIC, seed=9, tensor_id=4, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    dx = oracle.bf16_round(oracle.gemm_dgrad(dequant_from_gpu(qdy), dequant_from_gpu(qw)))
    dx_bits = workloads.bf16_bits(torch.from_numpy(dx).to(torch.bfloat16))
    o_rm, o_t, o_s = oracle.quantize2d(dx_bits, oracle.MODE_STOCHASTIC, 9, 4)
    compare_logical(dxq, o_rm, o_t, o_s, T, K)


@pytest.mark.parametrize("mode", [0, 1])
def test_grouped_fused_products_equal_product_then_quantize(mode):
    """The quantizing epilogue on grouped (mixture-of-experts) products, groups padded to 256 rows: forward and input
    gradient against the plain grouped product followed by fp4q_quantize2d, bit for bit."""
    E, H, F = 5, 256, 192
    counts = np.array([130, 0, 1, 300, 128])
    offs = workloads.padded_row_offsets(counts, 256)
    T = int(offs[-1])
    g = torch.Generator(device="cuda").manual_seed(21)
    X = workloads.zero_padding_rows(torch.randn(T, H, generator=g, device="cuda").to(torch.bfloat16), counts, offs)
    dY = workloads.zero_padding_rows((torch.randn(T, F, generator=g, device="cuda") * 0.01).to(torch.bfloat16), counts, offs)
    W = (torch.randn(E * F, H, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    qx, qw = binding.fp4q_quantize2d(X), binding.fp4q_quantize2d(W)
    qdy = binding.fp4q_quantize2d(dY, mode=1, seed=4, tensor_id=2)
    d_offs = torch.from_numpy(offs).cuda()
    ws = binding.alloc_workspace("cuda")
    fused_y = binding.fp4q_gemm_fwd_quantized(qx, qw, mode=mode, seed=3, tensor_id=8, ws=ws, row_offsets=d_offs)
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_BF16, row_offsets=d_offs, ws=ws, row_alignment=256)
    chain_y = binding.fp4q_quantize2d(y.contiguous(), mode=mode, seed=3, tensor_id=8)
    fused_dx = binding.fp4q_gemm_dgrad_quantized(qdy, qw, mode=mode, seed=5, tensor_id=9, ws=ws, row_offsets=d_offs)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=binding.OUT_BF16, row_offsets=d_offs, ws=ws, row_alignment=256)
    chain_dx = binding.fp4q_quantize2d(dx.contiguous(), mode=mode, seed=5, tensor_id=9)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    compare_logical(fused_y, *logical(chain_y), T, F)
    compare_logical(fused_dx, *logical(chain_dx), T, H)
    offs128 = torch.from_numpy(workloads.padded_row_offsets(counts, 128)).cuda()
    with pytest.raises(binding.Fp4qError):      # the binding states 256-row alignment; the library refuses anything else
        g128 = binding._CGroups(E, 128, offs128.data_ptr())
        cx, cw, cy = qx.c_struct(), qw.c_struct(), fused_y.c_struct()
        import ctypes
        binding._check(binding.lib().fp4q_gemm_fwd_quantized(ctypes.byref(cx), ctypes.byref(cw), ctypes.byref(cy), 0, 0, 0,
                                                             ctypes.byref(g128), ws.data_ptr(), ws.numel(), None), "fwd_quantized")
