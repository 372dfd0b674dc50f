"""GPU parity: the block-scaled FP4 GEMMs (forward, dgrad, wgrad; dense and grouped) and the MXFP8
query/key projections against the CPU oracle, through the C ABI.

Tolerance (stated by the build target): relative Frobenius error <= 1e-3 and, per output row,
max |G - O| <= 1e-2 * ||O_row||_inf.  FP32 outputs are compared with the float64 oracle, BF16 outputs
with the oracle rounded to BF16.  The quantized operands themselves are checked bit for bit first, so a
GEMM mismatch can only come from the GEMM."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import assert_matches_oracle, dequant_from_gpu

pytestmark = pytest.mark.gpu


def check(got: torch.Tensor, ref: np.ndarray, what=""):
    g = got.double().cpu().numpy()
    if got.dtype == torch.bfloat16:
        ref = oracle.bf16_round(ref)
    assert g.shape == ref.shape, (g.shape, ref.shape)
    denom = np.linalg.norm(ref)
    rel = np.linalg.norm(g - ref) / denom if denom > 0 else np.abs(g).max()
    assert rel <= 1e-3, "%s: relative Frobenius error %.3e" % (what, rel)
    row_inf = np.abs(ref).max(axis=1, keepdims=True)
    assert (np.abs(g - ref) <= 1e-2 * row_inf + 1e-300).all(), "%s: per-row max-abs bound violated" % what
    return rel


def quantized(x, mode, seed, tid):
    """Quantize on the GPU (checked bit-exact against the oracle) and return (QTensor, dequantized float64)."""
    qt = assert_matches_oracle(x, mode, seed=seed, tensor_id=tid)
    return qt, dequant_from_gpu(qt)


def linear_layer_case(W, X, dY, seed, ws, dt_fwd=binding.OUT_BF16, modes=(1, 1, 1)):
    qw, wd = quantized(W, modes[0], seed, 0)
    qx, xd = quantized(X, modes[1], seed, 1)
    qdy, dyd = quantized(dY, modes[2], seed, 2)
    y = binding.fp4q_gemm_fwd(qx, qw, dt=dt_fwd, ws=ws)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=dt_fwd, ws=ws)
    dw = binding.fp4q_gemm_wgrad(qdy, qx, dt=binding.OUT_F32, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    check(y, oracle.gemm_fwd(xd, wd), "fwd")
    check(dx, oracle.gemm_dgrad(dyd, wd), "dgrad")
    check(dw, oracle.gemm_wgrad(dyd, xd), "wgrad")
    return qw, qx, qdy, wd, xd, dyd


@pytest.fixture(scope="module")
def ws():
    return binding.alloc_workspace("cuda")


@pytest.mark.parametrize("dt", [binding.OUT_BF16, binding.OUT_F32])
def test_tiny_linear_layer_all_three_products(ws, dt):
    # W 256x256, X 128x256 (outlier columns), dY 128x256; stochastic rounding, Philox seed 0
    t = workloads.tiny_layer("cuda")
    linear_layer_case(t["W"], t["X"], t["dY"], 0, ws, dt_fwd=dt)


def test_paper_faithful_rounding_modes(ws):
    # nearest for weights and activations (forward), stochastic for the output gradient (backward)
    t = workloads.tiny_layer("cuda")
    linear_layer_case(t["W"], t["X"], t["dY"], 7, ws, modes=(0, 0, 1))


def test_exact_case_grid_operands_fp32_bitwise(ws):
    # operands on the E2M1 grid times a power of two: every partial sum is exact in FP32, so the GPU
    # result must equal the oracle bit for bit whatever the accumulation order
    g = torch.Generator(device="cuda").manual_seed(1)
    grid = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6], device="cuda")
    def draw(r, c, e):
        v = grid[torch.randint(0, 8, (r, c), generator=g, device="cuda")]
        s = torch.randint(0, 2, (r, c), generator=g, device="cuda") * 2 - 1
        return (v * s * 2.0 ** e).to(torch.bfloat16)
    X, W, dY = draw(256, 512, -3), draw(384, 512, 5), draw(256, 384, 2)
    qx, xd = quantized(X, 0, 0, 0)
    qw, wd = quantized(W, 0, 0, 1)
    qdy, dyd = quantized(dY, 0, 0, 2)
    assert np.array_equal(xd, X.double().cpu().numpy())
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_F32, ws=ws)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=binding.OUT_F32, ws=ws)
    dw = binding.fp4q_gemm_wgrad(qdy, qx, dt=binding.OUT_F32, ws=ws)
    assert np.array_equal(y.double().cpu().numpy(), oracle.gemm_fwd(xd, wd))
    assert np.array_equal(dx.double().cpu().numpy(), oracle.gemm_dgrad(dyd, wd))
    assert np.array_equal(dw.double().cpu().numpy(), oracle.gemm_wgrad(dyd, xd))


def test_scale_layout_probe_distinct_scale_per_block(ws):
    # every 32x32 block of every operand gets its own power-of-two magnitude: a scale byte replicated to
    # the wrong row or contraction block changes the result by a factor >= 2
    g = torch.Generator(device="cuda").manual_seed(2)
    def spread(r, c, a, b, m):
        i = torch.arange(r, device="cuda")[:, None] // 32
        j = torch.arange(c, device="cuda")[None, :] // 32
        return (torch.randn(r, c, generator=g, device="cuda") * torch.exp2(((a * i + b * j) % m).float() - m // 2)).to(torch.bfloat16)
    X, W, dY = spread(384, 640, 1, 2, 11), spread(512, 640, 3, 1, 13), spread(384, 512, 2, 3, 7)
    linear_layer_case(W, X, dY, 3, ws, dt_fwd=binding.OUT_F32)


@pytest.mark.parametrize("T,N,K", [(100, 200, 96), (129, 257, 160), (1, 8, 32), (300, 72, 1000), (64, 520, 288)])
def test_ragged_shapes(ws, T, N, K):
    # sizes that are not multiples of the 128x256 tile, the 256-element stage or the 32-element block
    g = torch.Generator(device="cuda").manual_seed(T + N + K)
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    X = torch.randn(T, K, generator=g, device="cuda").to(torch.bfloat16)
    dY = (torch.randn(T, N, generator=g, device="cuda") * 1e-3).to(torch.bfloat16)
    linear_layer_case(W, X, dY, 5, ws, dt_fwd=binding.OUT_BF16 if (T + N) % 2 else binding.OUT_F32)


def test_multi_tile_long_contraction_and_accumulate(ws):
    # several tiles per CTA (persistent loop), ring wrap-around, ragged tail, and dW += in FP32
    cfg = workloads.CONFIG_1B
    lay = ("down", 1152, 2304)
    t = workloads.dense_layer_tensors(cfg, lay, 6, "cuda", tokens=1000)
    qw, qx, qdy, wd, xd, dyd = linear_layer_case(t["W"], t["X"], t["dY"], cfg.philox_seed, ws)
    base = torch.randn(1152, 2304, device="cuda")
    acc = base.clone()
    binding.fp4q_gemm_wgrad(qdy, qx, out=acc, dt=binding.OUT_F32, accumulate=True, ws=ws)
    check(acc, base.double().cpu().numpy() + oracle.gemm_wgrad(dyd, xd), "wgrad accumulate")


def test_full_size_7b_shapes_sampled_rows(ws):
    # 7B-class gate projection at full size (T=16384, N=11008, K=4096) in the benchmark's launch
    # configuration; the oracle recomputes a deterministic row sample (first, last, 62 seeded rows)
    cfg = workloads.CONFIG_7B
    lay = cfg.layers()[4]
    t = workloads.dense_layer_tensors(cfg, lay, 4, "cuda")
    qw = binding.fp4q_quantize2d(t["W"], mode=1, seed=cfg.philox_seed, tensor_id=40)
    qx = binding.fp4q_quantize2d(t["X"], mode=1, seed=cfg.philox_seed, tensor_id=41)
    qdy = binding.fp4q_quantize2d(t["dY"], mode=1, seed=cfg.philox_seed, tensor_id=42)
    y = binding.fp4q_gemm_fwd(qx, qw, ws=ws)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, ws=ws)
    dw = binding.fp4q_gemm_wgrad(qdy, qx, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    wd, xd, dyd = dequant_from_gpu(qw), None, None
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, cfg.tokens - 1], rng.integers(0, cfg.tokens, 62)]))
    def deq_rows(qt, rows):
        # dequantize whole 32-row blocks that contain the sampled rows, then pick the rows
        out = []
        for r in rows:
            b = r // 32
            q = qt.q_rm[32 * b:32 * b + 32, :(qt.cols + 1) // 2].cpu().numpy()
            s = qt.scale[b:b + 1].cpu().numpy()
            out.append(oracle.dequantize2d(np.ascontiguousarray(q), np.ascontiguousarray(s), 32, qt.cols)[r % 32])
        return np.stack(out)
    xs, dys = deq_rows(qx, rows), deq_rows(qdy, rows)
    check(y[torch.from_numpy(rows).cuda()], oracle.gemm_fwd(xs, wd), "fwd 7B sample")
    check(dx[torch.from_numpy(rows).cuda()], oracle.gemm_dgrad(dys, wd), "dgrad 7B sample")
    # wgrad: sample output rows n; needs all tokens of the sampled dY columns
    ncols = np.unique(np.concatenate([[0, lay[1] - 1], rng.integers(0, lay[1], 14)]))
    xd = dequant_from_gpu(qx)
    dyd_cols = np.stack([_deq_col(qdy, int(c)) for c in ncols], axis=1)
    check(dw[torch.from_numpy(ncols).cuda()], dyd_cols.T @ xd, "wgrad 7B sample")


def _deq_col(qt, c):
    """One column of the dequantized tensor from the transposed payload (exercises q_t as well)."""
    q = qt.q_t[c, :(qt.rows + 1) // 2].cpu().numpy()
    codes = np.empty(qt.rows, dtype=np.uint8)
    codes[0::2] = q & 0xF
    codes[1::2] = q >> 4
    vals = np.array([oracle.e2m1_value(int(k)) for k in range(16)])[codes]
    s = qt.scale[:, c // 32].cpu().numpy().astype(np.int64)
    return vals * np.ldexp(1.0, np.repeat(s, 32)[:qt.rows] - 127)


# ----------------------------------------------------------------------------------------- grouped (MoE)

def _moe_case(ws, E, H, F, counts, seed, pad=128):
    offs = workloads.padded_row_offsets(counts, pad)
    T = int(offs[-1])
    g = torch.Generator(device="cuda").manual_seed(seed)
    X = workloads.zero_padding_rows(torch.randn(T, H, generator=g, device="cuda").to(torch.bfloat16), counts, offs)
    dY = workloads.zero_padding_rows((torch.randn(T, F, generator=g, device="cuda") * 0.01).to(torch.bfloat16), counts, offs)
    W = (torch.randn(E * F, H, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    qx, xd = quantized(X, 1, seed, 1)
    qw, wd = quantized(W, 1, seed, 0)
    qdy, dyd = quantized(dY, 1, seed, 2)
    d_offs = torch.from_numpy(offs).cuda()
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_BF16, row_offsets=d_offs, ws=ws, row_alignment=pad)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=binding.OUT_BF16, row_offsets=d_offs, ws=ws, row_alignment=pad)
    dw = binding.fp4q_gemm_wgrad(qdy, qx, dt=binding.OUT_F32, row_offsets=d_offs, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    check(y, oracle.grouped(oracle.gemm_fwd, xd, wd, offs), "grouped fwd")
    check(dx, oracle.grouped(oracle.gemm_dgrad, dyd, wd, offs), "grouped dgrad")
    ref_dw = oracle.grouped_wgrad(dyd, xd, offs)
    got = dw.double().cpu().numpy()
    for e in range(E):                      # per expert, so that a tiny expert is not hidden by a big one
        blk = slice(e * F, (e + 1) * F)
        if counts[e] == 0:
            assert not got[blk].any()
        else:
            check(dw[blk], ref_dw[blk], "grouped wgrad expert %d" % e)


def test_grouped_small_with_empty_and_uneven_groups(ws):
    _moe_case(ws, E=5, H=256, F=192, counts=np.array([130, 0, 1, 300, 128]), seed=11)


def test_grouped_expert_width_not_a_multiple_of_the_tile_and_accumulation(ws):
    # expert width 320: in the weight gradient's second pair tile the first CTA holds 64 valid rows and the second none;
    # the rows below belong to the next expert's block of the output and must stay untouched; then the same product
    # accumulated into FP32
    E, H, F = 3, 320, 320
    counts = np.array([64, 200, 0])
    _moe_case(ws, E=E, H=H, F=F, counts=counts, seed=13)
    offs = workloads.padded_row_offsets(counts, 128)
    T = int(offs[-1])
    g = torch.Generator(device="cuda").manual_seed(14)
    X = workloads.zero_padding_rows(torch.randn(T, H, generator=g, device="cuda").to(torch.bfloat16), counts, offs)
    dY = workloads.zero_padding_rows((torch.randn(T, F, generator=g, device="cuda") * 0.01).to(torch.bfloat16), counts, offs)
    qx, xd = quantized(X, 0, 1, 1)
    qdy, dyd = quantized(dY, 1, 1, 2)
    acc = torch.full((E * F, H), 0.5, dtype=torch.float32, device="cuda")
    binding.fp4q_gemm_wgrad(qdy, qx, out=acc, dt=binding.OUT_F32, accumulate=True, row_offsets=torch.from_numpy(offs).cuda(), ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    ref = oracle.grouped_wgrad(dyd, xd, offs) + 0.5
    got = acc.double().cpu().numpy()
    assert np.array_equal(got[2 * F:], np.full((F, H), 0.5))      # the empty expert adds nothing
    check(acc[:2 * F], ref[:2 * F], "grouped wgrad, accumulate")


def test_grouped_with_groups_aligned_to_256_rows_runs_on_pairs(ws):
    # the caller states that every group starts on a multiple of 256 rows: forward and input gradient then use the
    # 256-row pair tiles; empty, tiny and uneven groups as above
    _moe_case(ws, E=5, H=256, F=192, counts=np.array([130, 0, 1, 300, 128]), seed=15, pad=256)
    cfg = workloads.CONFIG_MOE
    counts = workloads.moe_routing(cfg, tokens=1024, experts=8)
    _moe_case(ws, E=8, H=cfg.hidden, F=cfg.expert_ffn, counts=counts, seed=16, pad=256)


def test_grouped_moe_shapes_reduced_expert_count(ws):
    # expert-layer shapes of the MoE configuration (hidden 2048, expert FFN 768), Zipf(1.2) top-8 loads,
    # on 16 experts and 2048 tokens so that the oracle finishes in seconds
    cfg = workloads.CONFIG_MOE
    counts = workloads.moe_routing(cfg, tokens=2048, experts=16)
    assert counts.sum() == 2048 * cfg.top_k
    _moe_case(ws, E=16, H=cfg.hidden, F=cfg.expert_ffn, counts=counts, seed=cfg.philox_seed)


# ----------------------------------------------------------------------------------------- MXFP8 Q/K

def _mxfp8_operand(x):
    q, s = binding.fp4q_mxfp8_quantize1d(x)
    torch.cuda.synchronize()
    oq, os_ = oracle.mxfp8_quantize1d(workloads.bf16_bits(x))
    rows, cols = x.shape
    gq = q.cpu().numpy()
    assert np.array_equal(gq[:, :cols], oq), "MXFP8 payload differs"
    assert not gq[:, cols:].any()
    assert np.array_equal(s.cpu().numpy(), os_), "MXFP8 scales differ"
    return q, s, oracle.mxfp8_dequantize(oq, os_)


@pytest.mark.parametrize("T,N,K", [(128, 256, 256), (200, 136, 416), (512, 768, 1024)])
def test_mxfp8_qk_projections(ws, T, N, K):
    g = torch.Generator(device="cuda").manual_seed(T + K)
    X = workloads.activations_student_t(T, K, 400 + T, "cuda", nu=3)
    Wq = (torch.randn(N, K, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    Wk = (torch.randn(N, K, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    xq, xs, xd = _mxfp8_operand(X)
    wqq, wqs, wqd = _mxfp8_operand(Wq)
    wkq, wks, wkd = _mxfp8_operand(Wk)
    for dt in (binding.OUT_BF16, binding.OUT_F32):
        q_out, k_out = binding.fp4q_mxfp8_qk(xq, xs, wqq, wqs, wkq, wks, T, K, N, dt=dt, ws=ws)
        torch.cuda.synchronize()
        assert binding.fp4q_workspace_status(ws) == 0
        check(q_out, oracle.gemm_fwd(xd, wqd), "Q projection")
        check(k_out, oracle.gemm_fwd(xd, wkd), "K projection")


def test_mxfp8_quantize_edge_values():
    bits = np.zeros((4, 96), dtype=np.uint16)
    bits[0, :32] = 0x43E0                      # 448 everywhere: scale 1
    bits[0, 32] = 0x43E1                       # just above 448: scale 2
    bits[1, :] = np.arange(96) | 0x3F00
    bits[2, 5], bits[2, 6], bits[2, 7] = 0x7F80, 0xFF80, 0x7FC0    # +Inf, -Inf, NaN
    bits[3, :64] = np.arange(64)               # subnormals
    _mxfp8_operand(workloads.bits_to_bf16(bits, "cuda"))
    _mxfp8_operand(workloads.activations_student_t(70, 200, 9, "cuda", nu=3))   # ragged columns


def test_one_cta_kernel_for_dense_products():
    """Dense FP4 products default to cta_group::2 pairs; FP4Q_CTA_PAIRS=0 (read once per process) selects the
    one-CTA kernel.  The dense parity cases are repeated in a child process with that switch."""
    import os
    import subprocess
    import sys
    if os.environ.get("FP4Q_CTA_PAIRS") == "0":
        pytest.skip("already running with the one-CTA kernel")
    env = dict(os.environ, FP4Q_CTA_PAIRS="0")
    here = os.path.dirname(os.path.abspath(__file__))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(here, "test_gpu_gemm.py"), "-m", "gpu", "-q", "-x",
                        "-k", "tiny_linear or ragged or exact_case or scale_layout or multi_tile"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_group_descriptor_is_validated(ws):
    x = workloads.weights(256, 64, 1, "cuda")
    w = workloads.weights(64, 64, 2, "cuda")
    qx, qw = binding.fp4q_quantize2d(x), binding.fp4q_quantize2d(w)
    offs = torch.tensor([0, 256], dtype=torch.int64, device="cuda")
    with pytest.raises(binding.Fp4qError):
        binding.fp4q_gemm_fwd(qx, qw, row_offsets=offs, ws=ws, row_alignment=64)     # only 0, 128 and 256 are statements the library knows
    y = binding.fp4q_gemm_fwd(qx, qw, row_offsets=offs, ws=ws, row_alignment=256)
    y0 = binding.fp4q_gemm_fwd(qx, qw, ws=ws)
    torch.cuda.synchronize()
    assert torch.equal(y, y0)                                                       # one group = the dense product


def test_seeded_random_shapes_all_three_products(ws):
    # two dozen seeded shapes around the tile edges (one CTA / pairs, ragged rows, columns and contraction tails)
    rng = np.random.default_rng(2024)
    for n in range(24):
        T = int(rng.choice([1, 31, 64, 127, 128, 129, 255, 256, 257, 300, 513, 640]))
        N = int(rng.choice([8, 32, 96, 200, 256, 264, 512, 520, 768]))
        K = int(rng.choice([32, 64, 96, 256, 288, 1000, 1024, 2080]))
        g = torch.Generator(device="cuda").manual_seed(1000 + n)
        W = (torch.randn(N, K, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
        X = torch.randn(T, K, generator=g, device="cuda").to(torch.bfloat16)
        dY = (torch.randn(T, N, generator=g, device="cuda") * 1e-3).to(torch.bfloat16)
        linear_layer_case(W, X, dY, seed=n, ws=ws, dt_fwd=binding.OUT_BF16 if n & 1 else binding.OUT_F32)


def test_seeded_random_grouped_cases(ws):
    # random expert counts (empty experts included), widths and paddings; both paddings run (pairs with 256)
    rng = np.random.default_rng(77)
    for n in range(8):
        E = int(rng.integers(1, 7))
        counts = rng.integers(0, 400, size=E)
        counts[rng.integers(0, E)] = 0 if E > 1 else counts[0]
        H = int(rng.choice([64, 256, 320, 1024]))
        F = int(rng.choice([64, 128, 192, 448]))
        _moe_case(ws, E=E, H=H, F=F, counts=counts, seed=200 + n, pad=128 if n & 1 else 256)
