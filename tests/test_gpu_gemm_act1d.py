"""GPU parity of the products with the paper's mixed layout (Section 3.1: 2D blocks for weights and gradients, 1D
blocks for activations): Y = X^ W^^T with X in 1D blocks along the channels, and dW = dY^^T X^_t with X re-quantized
in 1D blocks along the tokens.  Operands are quantized on the GPU (bit-exactness is covered elsewhere and re-checked
here), the expected products come from the oracle's dequantized operands in float64."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import assert_matches_oracle, dequant_from_gpu

pytestmark = pytest.mark.gpu


def check(got, ref, what):
    g = got.double().cpu().numpy()
    if got.dtype == torch.bfloat16:
        ref = oracle.bf16_round(ref)
    rel = np.linalg.norm(g - ref) / np.linalg.norm(ref)
    assert rel <= 1e-3, "%s: relative Frobenius error %.3e" % (what, rel)
    row_inf = np.abs(ref).max(axis=1, keepdims=True)
    assert (np.abs(g - ref) <= 1e-2 * row_inf + 1e-300).all(), "%s: per-row max-abs bound violated" % what


def act1d(x):
    """Row-wise 1D encoding from the GPU, checked against the oracle; returns (q, s, dequantized [T, K])."""
    rows, cols = x.shape
    q, s = binding.fp4q_quantize1d(x)
    torch.cuda.synchronize()
    oq, os_ = oracle.quantize1d(workloads.bf16_bits(x))
    assert np.array_equal(q.cpu().numpy()[:, :oq.shape[1]], oq) and np.array_equal(s.cpu().numpy()[:, :os_.shape[1]], os_)
    return q, s, oracle.dequantize1d(oq, os_, rows, cols)


def act1d_t(x):
    """Transposed 1D encoding from the GPU, checked; returns (q, s, dequantized as [T, K])."""
    rows, cols = x.shape
    q, s = binding.fp4q_quantize1d_t(x)
    torch.cuda.synchronize()
    oq, os_ = oracle.quantize1d_t(workloads.bf16_bits(x))
    assert np.array_equal(q.cpu().numpy()[:, :oq.shape[1]], oq) and np.array_equal(s.cpu().numpy()[:, :os_.shape[1]], os_)
    return q, s, oracle.dequantize1d(oq, os_, cols, rows).T


SHAPES = [(128, 256, 256),      # one tile (one-CTA kernel)
          (384, 512, 1280),     # pairs, several units of four stages, ragged last unit
          (200, 300, 416),      # ragged in every dimension (K tail inside an MMA)
          (1024, 768, 2048)]    # several tiles per CTA


@pytest.mark.parametrize("T,N,K", SHAPES)
@pytest.mark.parametrize("dt", [binding.OUT_BF16, binding.OUT_F32])
def test_forward_with_1d_activations(T, N, K, dt):
    x = workloads.activations_gauss_outliers(T, K, seed=1, device="cuda")
    w = workloads.weights(N, K, seed=2, device="cuda")
    xq, xs, x_hat = act1d(x)
    W = assert_matches_oracle(w, binding.ROUND_NEAREST, seed=0, tensor_id=0)
    y = binding.fp4q_gemm_fwd_act1d(xq, xs, T, W, dt=dt)
    torch.cuda.synchronize()
    check(y, oracle.gemm_fwd(x_hat, dequant_from_gpu(W)), "forward, 1D activations")


@pytest.mark.parametrize("T,N,K", SHAPES)
def test_wgrad_with_1d_activations(T, N, K):
    x = workloads.activations_gauss_outliers(T, K, seed=3, device="cuda")
    dy = workloads.gradients_rowscaled(T, N, seed=4, device="cuda")
    xtq, xts, x_hat_t = act1d_t(x)
    dY = assert_matches_oracle(dy, binding.ROUND_STOCHASTIC, seed=7, tensor_id=2)
    dw = binding.fp4q_gemm_wgrad_act1d(dY, xtq, xts, K, dt=binding.OUT_F32)
    torch.cuda.synchronize()
    ref = oracle.gemm_wgrad(dequant_from_gpu(dY), x_hat_t)
    check(dw, ref, "wgrad, 1D activations")
    # accumulation into an FP32 gradient buffer
    acc = torch.full((N, K), 0.25, dtype=torch.float32, device="cuda")
    binding.fp4q_gemm_wgrad_act1d(dY, xtq, xts, K, out=acc, dt=binding.OUT_F32, accumulate=True)
    torch.cuda.synchronize()
    check(acc, ref + 0.25, "wgrad, 1D activations, accumulate")


def test_mixed_layout_differs_from_all_2d_and_shows_the_inconsistency():
    """The two 1D encodings of one activation dequantize to different tensors (Figure 1), the 2D ones do not; and the
    1D forward product is not the all-2D product (the kernel really reads per-row scales)."""
    T, N, K = 256, 256, 512
    x = workloads.activations_gauss_outliers(T, K, seed=5, device="cuda")
    w = workloads.weights(N, K, seed=6, device="cuda")
    xq, xs, x_fwd = act1d(x)
    _, _, x_bwd = act1d_t(x)
    assert np.linalg.norm(x_fwd - x_bwd) / np.linalg.norm(x_fwd) > 1e-2
    W = binding.fp4q_quantize2d(w)
    X2 = binding.fp4q_quantize2d(x)
    y1 = binding.fp4q_gemm_fwd_act1d(xq, xs, T, W, dt=binding.OUT_F32)
    y2 = binding.fp4q_gemm_fwd(X2, W, dt=binding.OUT_F32)
    torch.cuda.synchronize()
    assert (y1 - y2).norm() / y2.norm() > 1e-3


def test_full_size_attention_projection_sampled_rows():
    """16384 tokens, 4096 x 4096 (the shape the benchmark times these products on), in the benchmark's launch
    configuration: the oracle recomputes a deterministic sample of output rows from operands it dequantizes itself."""
    T, N, K = 16384, 4096, 4096
    x = workloads.activations_student_t(T, K, 21, "cuda")
    w = workloads.weights(N, K, 22, "cuda")
    dy = workloads.gradients_rowscaled(T, N, 23, "cuda")
    W = binding.fp4q_quantize2d(w)
    dY = binding.fp4q_quantize2d(dy, mode=1, seed=5, tensor_id=2)
    xq, xs = binding.fp4q_quantize1d(x)
    xtq, xts = binding.fp4q_quantize1d_t(x)
    ws = binding.alloc_workspace("cuda")
    y = binding.fp4q_gemm_fwd_act1d(xq, xs, T, W, dt=binding.OUT_F32, ws=ws)
    dw = binding.fp4q_gemm_wgrad_act1d(dY, xtq, xts, K, dt=binding.OUT_F32, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([[0, T - 1], rng.integers(0, T, 30)]))
    # forward: sampled token rows; the oracle quantizes those rows itself (1D blocks lie inside a row)
    oq, os_ = oracle.quantize1d(workloads.bf16_bits(x[torch.from_numpy(rows).cuda()]))
    g_q = xq[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert np.array_equal(g_q[:, :oq.shape[1]], oq)
    x_hat = oracle.dequantize1d(oq, os_, len(rows), K)
    check(y[torch.from_numpy(rows).cuda()], oracle.gemm_fwd(x_hat, dequant_from_gpu(W)), "forward sample, 1D activations")
    # weight gradient: sampled output rows n need column n of dY over all tokens and the whole transposed encoding of X
    ncols = np.unique(np.concatenate([[0, N - 1], rng.integers(0, N, 10)]))
    dyd = dequant_from_gpu(dY)[:, ncols]
    xt_hat = oracle.dequantize1d(np.ascontiguousarray(xtq.cpu().numpy()[:, :T // 2]), np.ascontiguousarray(xts.cpu().numpy()), K, T)
    sample_cols = rng.integers(0, K, 16)           # the transposed encoding itself, on sampled columns of x
    oq_t, os_t = oracle.quantize1d(np.ascontiguousarray(workloads.bf16_bits(x[:, torch.from_numpy(sample_cols).cuda()]).T))
    assert np.array_equal(xtq.cpu().numpy()[sample_cols, :T // 2], oq_t) and np.array_equal(xts.cpu().numpy()[sample_cols], os_t)
    check(dw[torch.from_numpy(ncols).cuda()], dyd.T @ xt_hat.T, "wgrad sample, 1D activations")


def test_seeded_random_shapes_with_1d_activations():
    rng = np.random.default_rng(31)
    ws = binding.alloc_workspace("cuda")
    for n in range(10):
        T = int(rng.choice([1, 96, 128, 129, 256, 300, 513]))
        N = int(rng.choice([32, 200, 256, 264, 512]))
        K = int(rng.choice([32, 96, 256, 288, 1000, 1024, 2080]))
        x = workloads.activations_gauss_outliers(T, K, seed=40 + n, device="cuda")
        w = workloads.weights(N, K, seed=60 + n, device="cuda")
        dy = workloads.gradients_rowscaled(T, N, seed=80 + n, device="cuda")
        xq, xs, x_hat = act1d(x)
        xtq, xts, x_hat_t = act1d_t(x)
        W = assert_matches_oracle(w, binding.ROUND_NEAREST, seed=0, tensor_id=0)
        dY = assert_matches_oracle(dy, binding.ROUND_STOCHASTIC, seed=n, tensor_id=2)
        y = binding.fp4q_gemm_fwd_act1d(xq, xs, T, W, dt=binding.OUT_BF16 if n & 1 else binding.OUT_F32, ws=ws)
        dw = binding.fp4q_gemm_wgrad_act1d(dY, xtq, xts, K, dt=binding.OUT_F32, ws=ws)
        torch.cuda.synchronize()
        assert binding.fp4q_workspace_status(ws) == 0
        check(y, oracle.gemm_fwd(x_hat, dequant_from_gpu(W)), "forward, 1D activations, shape %d" % n)
        check(dw, oracle.gemm_wgrad(dequant_from_gpu(dY), x_hat_t), "wgrad, 1D activations, shape %d" % n)
