"""GPU parity at the stated shapes of the benchmark configurations that the small cases do not reach: the
1B-class dense layers (8192 tokens), the MXFP8 query/key projections at 7B shapes (16384 x 4096 x 4096) and
the 128-expert mixture-of-experts layer (16384 tokens, top-8, Zipf(1.2) loads), all in the launch
configuration the benchmark times.

The kernels run on the whole problem; the oracle recomputes what it can finish in seconds: whole products
where they are small enough, otherwise a deterministic sample of output rows (first and last row of the
matrix and of every token group, plus seeded random rows - all columns of each), and for the grouped weight
gradient whole experts (the largest, the smallest, an empty one and two seeded ones).  Quantized operands are
compared bit for bit on sampled block rows first; the products are then computed by the oracle from the
GPU's own payloads (decoded with the oracle's decoder), so a mismatch can only come from the GEMM."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import HostQ, assert_windows_match_oracle, check_gemm

pytestmark = pytest.mark.gpu

SR = binding.ROUND_STOCHASTIC


@pytest.fixture(scope="module")
def ws():
    return binding.alloc_workspace("cuda")


def _sample_rows(n_rows, n_random, seed):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([[0, n_rows - 1], rng.integers(0, n_rows, n_random)]))


# ----------------------------------------------------------------------------------------- 1B-class dense layers

@pytest.mark.parametrize("index", [0, 4, 6])   # q (2048 x 2048), gate (5632 x 2048), down (2048 x 5632)
def test_dense_1b_layers_at_8192_tokens(ws, index):
    cfg = workloads.CONFIG_1B
    lay = cfg.layers()[index]
    _, N, K = lay
    t = workloads.dense_layer_tensors(cfg, lay, index, "cuda")
    q = {}
    for tid, name in enumerate(["W", "X", "dY"]):
        q[name] = binding.fp4q_quantize2d(t[name], mode=SR, seed=cfg.philox_seed, tensor_id=10 * index + tid)
        n_blk = (t[name].shape[0] + 31) // 32
        assert_windows_match_oracle(t[name], q[name], [0, n_blk - 1, (7 * index + 3) % n_blk], SR, cfg.philox_seed,
                                    10 * index + tid)
    y = binding.fp4q_gemm_fwd(q["X"], q["W"], ws=ws)
    dx = binding.fp4q_gemm_dgrad(q["dY"], q["W"], ws=ws)
    dw = binding.fp4q_gemm_wgrad(q["dY"], q["X"], ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    hw, hx, hdy = HostQ(q["W"]), HostQ(q["X"]), HostQ(q["dY"])
    wd = hw.row_range(0, N)
    if index == 0:
        # the square layer in full: every output element of all three products
        xd, dyd = hx.row_range(0, cfg.tokens), hdy.row_range(0, cfg.tokens)
        check_gemm(y, oracle.gemm_fwd(xd, wd), "fwd 1B q, full")
        check_gemm(dx, oracle.gemm_dgrad(dyd, wd), "dgrad 1B q, full")
        check_gemm(dw, oracle.gemm_wgrad(dyd, xd), "wgrad 1B q, full")
        return
    rows = _sample_rows(cfg.tokens, 254, index)
    ridx = torch.from_numpy(rows).cuda()
    check_gemm(y[ridx], oracle.gemm_fwd(hx.take_rows(rows), wd), "fwd 1B %s, %d rows" % (lay[0], len(rows)))
    check_gemm(dx[ridx], oracle.gemm_dgrad(hdy.take_rows(rows), wd), "dgrad 1B %s, %d rows" % (lay[0], len(rows)))
    out_rows = _sample_rows(N, 30, 100 + index)               # rows of dW = columns of dY, over all tokens
    dyc = hdy.take_cols(out_rows)
    check_gemm(dw[torch.from_numpy(out_rows).cuda()], dyc.T @ hx.row_range(0, cfg.tokens), "wgrad 1B %s, %d rows" % (lay[0], len(out_rows)))


# ----------------------------------------------------------------------------------------- MXFP8 Q/K at 7B shapes

def test_mxfp8_qk_projections_at_7b_shapes(ws):
    cfg = workloads.CONFIG_ATTN_7B
    T, H = cfg.tokens, cfg.hidden
    X = workloads.activations_student_t(T, H, cfg.data_seed + 1, "cuda", nu=cfg.nu)
    Wq = workloads.weights(H, H, cfg.data_seed, "cuda")
    Wk = workloads.weights(H, H, cfg.data_seed + 10, "cuda")
    xq, xs = binding.fp4q_mxfp8_quantize1d(X)
    wqq, wqs = binding.fp4q_mxfp8_quantize1d(Wq)
    wkq, wks = binding.fp4q_mxfp8_quantize1d(Wk)
    q_out, k_out = binding.fp4q_mxfp8_qk(xq, xs, wqq, wqs, wkq, wks, T, H, H, dt=binding.OUT_BF16, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    # operands: both weights in full, the activation on the sampled rows (1 x 32 blocks: rows are independent)
    rows = _sample_rows(T, 126, 4)
    ridx = torch.from_numpy(rows).cuda()
    o_xq, o_xs = oracle.mxfp8_quantize1d(workloads.bf16_bits(X[ridx]))
    assert np.array_equal(xq[ridx].cpu().numpy(), o_xq) and np.array_equal(xs[ridx].cpu().numpy(), o_xs)
    xd = oracle.mxfp8_dequantize(o_xq, o_xs)
    for name, W, wq, wsc, out in (("Q", Wq, wqq, wqs, q_out), ("K", Wk, wkq, wks, k_out)):
        o_wq, o_ws = oracle.mxfp8_quantize1d(workloads.bf16_bits(W))
        assert np.array_equal(wq.cpu().numpy(), o_wq), name
        assert np.array_equal(wsc.cpu().numpy(), o_ws), name
        check_gemm(out[ridx], oracle.gemm_fwd(xd, oracle.mxfp8_dequantize(o_wq, o_ws)), "%s projection, %d rows" % (name, len(rows)))


# ----------------------------------------------------------------------------------------- 128-expert MoE layer

def _moe_full_size_layer(ws, cfg, counts, pad, name, N, K, index):
    E = cfg.experts
    offs = workloads.padded_row_offsets(counts, pad)
    T = int(offs[-1])
    base = cfg.data_seed + 10 * index
    X = workloads.zero_padding_rows(workloads.activations_student_t(T, K, base + 1, "cuda"), counts, offs)
    dY = workloads.zero_padding_rows(workloads.gradients_rowscaled(T, N, base + 2, "cuda"), counts, offs)
    W = workloads.weights(E * N, K, base, "cuda")
    qw = binding.fp4q_quantize2d(W, mode=SR, seed=cfg.philox_seed, tensor_id=3 * index)
    qx = binding.fp4q_quantize2d(X, mode=SR, seed=cfg.philox_seed, tensor_id=3 * index + 1)
    qdy = binding.fp4q_quantize2d(dY, mode=SR, seed=cfg.philox_seed, tensor_id=3 * index + 2)
    # quantizer, bit for bit, on block rows at group boundaries: the block that holds a group's last valid row is
    # part data and part zero padding (boundary rule: only valid entries raise the block's maximum)
    ends = [(int(offs[g]) + int(counts[g]) - 1) // 32 for g in (0, E // 2, E - 1) if counts[g] > 0]
    assert_windows_match_oracle(X, qx, sorted(set([0, T // 32 - 1] + ends)), SR, cfg.philox_seed, 3 * index + 1)
    assert_windows_match_oracle(dY, qdy, sorted(set(ends)), SR, cfg.philox_seed, 3 * index + 2)
    assert_windows_match_oracle(W, qw, [0, (E * N) // 32 - 1, (E // 2 * N) // 32], SR, cfg.philox_seed, 3 * index)
    d_offs = torch.from_numpy(offs).cuda()
    y = binding.fp4q_gemm_fwd(qx, qw, row_offsets=d_offs, ws=ws, row_alignment=pad)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, row_offsets=d_offs, ws=ws, row_alignment=pad)
    dw = binding.fp4q_gemm_wgrad(qdy, qx, dt=binding.OUT_F32, row_offsets=d_offs, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    hw, hx, hdy = HostQ(qw), HostQ(qx), HostQ(qdy)
    # forward and input gradient: first and last valid row of every group, its last padding row, 512 seeded rows
    rng = np.random.default_rng(index)
    sample = {g: set() for g in range(E)}
    for g in range(E):
        r0, r1 = int(offs[g]), int(offs[g + 1])
        if counts[g] > 0:
            sample[g].update([r0, r0 + int(counts[g]) - 1])
        if r1 > r0:
            sample[g].add(r1 - 1)
    for r in rng.integers(0, T, 512):
        sample[int(np.searchsorted(offs, r, side="right") - 1)].add(int(r))
    n_checked = 0
    for g in range(E):
        rows = np.array(sorted(sample[g]), dtype=np.int64)
        if rows.size == 0:
            continue
        ridx = torch.from_numpy(rows).cuda()
        wd = hw.row_range(g * N, (g + 1) * N)
        check_gemm(y[ridx], oracle.gemm_fwd(hx.take_rows(rows), wd), "%s fwd, expert %d" % (name, g))
        check_gemm(dx[ridx], oracle.gemm_dgrad(hdy.take_rows(rows), wd), "%s dgrad, expert %d" % (name, g))
        pad_rows = rows[rows >= int(offs[g]) + int(counts[g])]
        if pad_rows.size:                                   # zero rows in, exact zeros out
            pidx = torch.from_numpy(pad_rows).cuda()
            assert not y[pidx].any() and not dx[pidx].any()
        n_checked += rows.size
    assert n_checked >= 512
    # weight gradient: whole experts
    nonempty = np.flatnonzero(counts > 0)
    experts = {int(nonempty[np.argmax(counts[nonempty])]), int(nonempty[np.argmin(counts[nonempty])]),
               int(rng.integers(0, E)), int(rng.integers(0, E))}
    experts.update(int(g) for g in np.flatnonzero(counts == 0)[:1])
    for g in sorted(experts):
        blk = dw[g * N:(g + 1) * N]
        if counts[g] == 0:
            assert not blk.any(), "empty expert %d" % g
            continue
        r0, r1 = int(offs[g]), int(offs[g + 1])
        check_gemm(blk, oracle.gemm_wgrad(hdy.row_range(r0, r1), hx.row_range(r0, r1)), "%s wgrad, expert %d (%d rows)" % (name, g, counts[g]))


@pytest.mark.parametrize("pad", [128, 256])
def test_moe_expert_layer_128_experts_16384_tokens(ws, pad):
    cfg = workloads.CONFIG_MOE
    counts = workloads.moe_routing(cfg)
    assert counts.size == 128 and counts.sum() == cfg.tokens * cfg.top_k
    if pad == 256:
        counts = counts.copy()
        counts[int(np.argmin(counts))] = 0        # one expert that no token chose
    # gate / up: 768 x 2048 per expert (contraction 2048); down: 2048 x 768 (contraction 768)
    _moe_full_size_layer(ws, cfg, counts, pad, "gate", cfg.expert_ffn, cfg.hidden, 0)
    _moe_full_size_layer(ws, cfg, counts, pad, "down", cfg.hidden, cfg.expert_ffn, 2)


def test_grouped_products_with_more_groups_than_the_shared_memory_tables_hold(ws):
    # 2900 groups of zero to three tokens, each non-empty one padded to 128 rows: more than 2048 row tiles and more than
    # 1023 groups exceed the per-tile group table and the boundary table, so every role looks its group up in global memory
    E, H, F = 2900, 64, 64
    rng = np.random.default_rng(5)
    counts = rng.integers(0, 4, size=E)
    counts[[0, E - 1]] = [3, 2]
    offs = workloads.padded_row_offsets(counts, 128)
    T = int(offs[-1])
    assert T // 128 > 2048
    g = torch.Generator(device="cuda").manual_seed(31)
    X = workloads.zero_padding_rows(torch.randn(T, H, generator=g, device="cuda").to(torch.bfloat16), counts, offs)
    dY = workloads.zero_padding_rows((torch.randn(T, F, generator=g, device="cuda") * 0.01).to(torch.bfloat16), counts, offs)
    W = (torch.randn(E * F, H, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    qx = binding.fp4q_quantize2d(X, mode=SR, seed=1, tensor_id=1)
    qw = binding.fp4q_quantize2d(W, mode=SR, seed=1, tensor_id=0)
    qdy = binding.fp4q_quantize2d(dY, mode=SR, seed=1, tensor_id=2)
    d_offs = torch.from_numpy(offs).cuda()
    y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_F32, row_offsets=d_offs, ws=ws)
    dx = binding.fp4q_gemm_dgrad(qdy, qw, dt=binding.OUT_F32, row_offsets=d_offs, ws=ws)
    dw = binding.fp4q_gemm_wgrad(qdy, qx, dt=binding.OUT_F32, row_offsets=d_offs, ws=ws)
    torch.cuda.synchronize()
    assert binding.fp4q_workspace_status(ws) == 0
    hw, hx, hdy = HostQ(qw), HostQ(qx), HostQ(qdy)
    xd, dyd, wd = hx.row_range(0, T), hdy.row_range(0, T), hw.row_range(0, E * F)
    check_gemm(y, oracle.grouped(oracle.gemm_fwd, xd, wd, offs), "grouped fwd, 2900 groups")
    check_gemm(dx, oracle.grouped(oracle.gemm_dgrad, dyd, wd, offs), "grouped dgrad, 2900 groups")
    ref = oracle.grouped_wgrad(dyd, xd, offs)
    got = dw.double().cpu().numpy()
    empty = np.repeat(counts == 0, F)
    assert not got[empty].any()
    check_gemm(dw[torch.from_numpy(np.flatnonzero(~empty)).cuda()], ref[~empty], "grouped wgrad, 2900 groups")
