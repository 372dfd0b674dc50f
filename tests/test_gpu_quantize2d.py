"""GPU parity: fp4q_quantize2d against the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_24953_b200 import binding, workloads
from tests.gpu_util import assert_matches_oracle, bits_tensor, gpu_quantize, logical

pytestmark = pytest.mark.gpu

MODES = [binding.ROUND_NEAREST, binding.ROUND_STOCHASTIC]


def _random_finite_bits(rng, rows, cols):
    b = rng.integers(0, 1 << 16, size=(rows, cols), dtype=np.uint32).astype(np.uint16)
    nonfinite = (b & 0x7F80) == 0x7F80
    b[nonfinite] &= 0xBFFF          # clear one exponent bit: finite
    return b


def _windowed_exponent_bits(rng, rows, cols):
    """Every 32x32 block gets its own exponent window so that all scale codes 0..253 occur."""
    b = rng.integers(0, 1 << 16, size=(rows, cols), dtype=np.uint32)
    rt, ct = rows // 32, cols // 32
    top = (np.arange(rt * ct) * 255 // (rt * ct)).reshape(rt, ct)          # biased exponent of the block maximum
    top = np.repeat(np.repeat(top, 32, 0), 32, 1)
    drop = rng.integers(0, 14, size=(rows, cols))
    be = np.clip(top - drop, 0, 254)
    return ((b & 0x807F) | (be << 7)).astype(np.uint16)


@pytest.mark.parametrize("mode", MODES)
def test_tiny_layer_config(mode):
    # W 256x256, X 128x256 with outlier columns, dY 128x256: Philox seed 0, tensor ids 0/1/2
    t = workloads.tiny_layer("cuda")
    for tid, name in enumerate(["W", "X", "dY"]):
        assert_matches_oracle(t[name], mode, seed=0, tensor_id=tid)


@pytest.mark.parametrize("mode", MODES)
def test_random_bit_patterns_and_all_scale_codes(mode):
    rng = np.random.default_rng(0)
    assert_matches_oracle(bits_tensor(_random_finite_bits(rng, 256, 384)), mode, seed=11, tensor_id=1)
    qt = assert_matches_oracle(bits_tensor(_windowed_exponent_bits(rng, 512, 512)), mode, seed=12, tensor_id=2)
    codes = set(np.unique(logical(qt)[2]).tolist())
    assert {0, 1, 2, 127, 240, 250, 253} <= codes or len(codes) > 200


@pytest.mark.parametrize("mode", MODES)
def test_exhaustive_ratio_sweep(mode):
    # every BF16 value v in [0, 6] (and its negative) against a block maximum of exactly 6, 6 - ulp,
    # 3 + ulp (just above a scale boundary) and 4: all rounding decisions of the format
    vals = np.array([b for b in range(0, 0x40C1)], dtype=np.uint16)          # 0 .. 6.0
    n = len(vals)
    for mx in (0x40C0, 0x40BF, 0x4041, 0x4080):
        per = 32 * 32 - 1
        blocks = -(-n // per)
        bits = np.zeros((32, 32 * blocks), dtype=np.uint16)
        for k in range(blocks):
            chunk = vals[k * per:(k + 1) * per]
            chunk = np.where(chunk <= mx, chunk, 0)
            tile = np.zeros(1024, dtype=np.uint16)
            tile[1:1 + len(chunk)] = chunk
            tile[0] = mx
            tile[1::2] |= 0x8000                                            # alternate signs
            bits[:, 32 * k:32 * k + 32] = tile.reshape(32, 32)
        assert_matches_oracle(bits_tensor(bits), mode, seed=5, tensor_id=9)


@pytest.mark.parametrize("shape", [(1, 1), (33, 31), (130, 200), (257, 129), (128, 144), (31, 1000)])
@pytest.mark.parametrize("mode", MODES)
def test_ragged_shapes(shape, mode):
    rng = np.random.default_rng(shape[0] * 7 + shape[1])
    x = (rng.standard_normal(shape) * np.exp(rng.standard_normal((shape[0], 1)) * 2)).astype(np.float32)
    assert_matches_oracle(torch.from_numpy(x).to(torch.bfloat16).cuda(), mode, seed=77, tensor_id=3)


@pytest.mark.parametrize("mode", MODES)
def test_strided_and_unaligned_input(mode):
    g = torch.Generator(device="cuda").manual_seed(4)
    big = torch.randn(300, 520, generator=g, device="cuda").to(torch.bfloat16)
    assert_matches_oracle(big[:, :512], mode, seed=1, tensor_id=1)          # ld_x != cols, aligned
    assert_matches_oracle(big[3:200, 1:385], mode, seed=1, tensor_id=1)     # 2-byte aligned only
    assert_matches_oracle(big[:, 8:264], mode, seed=1, tensor_id=1)         # 16-byte aligned offset


def test_transposition_invariance_on_gpu():
    # quantize(A)^T == quantize(A^T): scales transposed, row-major and transposed payloads swapped
    g = torch.Generator(device="cuda").manual_seed(6)
    a = (torch.randn(160, 96, generator=g, device="cuda") * 3).to(torch.bfloat16)
    at = a.t().contiguous()
    for mode, flags in ((binding.ROUND_NEAREST, 0), (binding.ROUND_STOCHASTIC, binding.INDEX_TRANSPOSED)):
        qa = logical(gpu_quantize(a, mode, seed=3, tensor_id=4))
        qb = logical(assert_matches_oracle(at, mode, seed=3, tensor_id=4, flags=flags))
        assert np.array_equal(qb[2], qa[2].T)
        assert np.array_equal(qb[0][:, :80], qa[1][:, :80]) and np.array_equal(qb[1][:, :48], qa[0][:, :48])


@pytest.mark.parametrize("mode", MODES)
def test_non_finite_inputs_have_defined_results(mode):
    rng = np.random.default_rng(9)
    bits = _random_finite_bits(rng, 64, 64) & 0xBFFF | 0x3000
    bits[0, 0], bits[0, 1], bits[5, 40], bits[40, 40] = 0x7F80, 0xFF80, 0x7FC0, 0xFFFF
    bits[33, 1:20] = 0x7F80
    assert_matches_oracle(bits_tensor(bits.astype(np.uint16)), mode, seed=2, tensor_id=2)


def test_without_transposed_payload_and_empty_inputs():
    g = torch.Generator(device="cuda").manual_seed(8)
    a = torch.randn(96, 64, generator=g, device="cuda").to(torch.bfloat16)
    assert_matches_oracle(a, binding.ROUND_STOCHASTIC, seed=1, want_t=False)
    for shape in [(0, 0), (0, 64), (64, 0)]:
        qt = binding.fp4q_quantize2d(torch.empty(shape, dtype=torch.bfloat16, device="cuda"))
        assert qt.rows == shape[0] and qt.cols == shape[1]


def test_deterministic_and_seed_sensitive():
    g = torch.Generator(device="cuda").manual_seed(10)
    a = torch.randn(256, 256, generator=g, device="cuda").to(torch.bfloat16)
    q1 = logical(gpu_quantize(a, binding.ROUND_STOCHASTIC, seed=123, tensor_id=1))
    q2 = logical(gpu_quantize(a, binding.ROUND_STOCHASTIC, seed=123, tensor_id=1))
    q3 = logical(gpu_quantize(a, binding.ROUND_STOCHASTIC, seed=124, tensor_id=1))
    q4 = logical(gpu_quantize(a, binding.ROUND_STOCHASTIC, seed=123, tensor_id=2))
    assert all(np.array_equal(x, y) for x, y in zip(q1, q2))
    assert not np.array_equal(q1[0], q3[0]) and not np.array_equal(q1[0], q4[0])
    assert np.array_equal(q1[2], q3[2])                                     # scales do not depend on the seed


def test_full_size_sampled_windows():
    # the 7B-class activation 16384x11008 in the launch configuration the benchmark times; the oracle
    # recomputes sampled windows of 2x3 blocks (corners, edges, seeded random positions)
    cfg = workloads.CONFIG_7B
    x = workloads.activations_student_t(cfg.tokens, cfg.ffn, cfg.data_seed + 61, "cuda", nu=cfg.nu)
    qt = gpu_quantize(x, binding.ROUND_STOCHASTIC, seed=cfg.philox_seed, tensor_id=7)
    rt, ct = cfg.tokens // 32, cfg.ffn // 32
    rng = np.random.default_rng(0)
    wins = [(0, 0), (rt - 2, ct - 3), (0, ct - 3), (rt - 2, 0)] + [(int(rng.integers(0, rt - 2)), int(rng.integers(0, ct - 3))) for _ in range(60)]
    for (I, J) in wins:
        rows = slice(32 * I, 32 * I + 64)
        sub_bits = None
        # the oracle needs the whole tensor only for its shape (the rounding stream is keyed on the
        # global element index), so hand it a view whose rows outside the window are never read
        full_rows = workloads.bf16_bits(x[rows])
        o_rm, o_t, o_s = _oracle_window(full_rows, cfg.tokens, cfg.ffn, I, J, cfg.philox_seed, 7)
        g_rm = qt.q_rm[32 * I:32 * I + 64, 16 * J:16 * J + 48].cpu().numpy()
        g_t = qt.q_t[32 * J:32 * J + 96, 16 * I:16 * I + 32].cpu().numpy()
        g_s = qt.scale[I:I + 2, J:J + 3].cpu().numpy()
        assert np.array_equal(g_s, o_s) and np.array_equal(g_rm, o_rm) and np.array_equal(g_t, o_t), (I, J)


def _oracle_window(rows_bits, total_rows, cols, I, J, seed, tid):
    """Run the oracle on block rows I..I+2, block columns J..J+3 of a [total_rows, cols] tensor given only
    the 64 rows that the window touches (placed at their true row offset in a sparse stand-in)."""
    import ctypes
    L = oracle.lib()
    q_rm = np.zeros((64, 48), dtype=np.uint8)
    q_t = np.zeros((96, 32), dtype=np.uint8)
    s = np.zeros((2, 3), dtype=np.uint8)
    # pointer arithmetic: pretend the tensor starts 32*I rows before the slice we hold
    base = rows_bits.ctypes.data - 32 * I * cols * 2
    rc = L.orc_quantize2d_window(ctypes.c_void_p(base), total_rows, cols, cols, oracle.MODE_STOCHASTIC, seed, tid, 0,
                                 I, I + 2, J, J + 3, q_rm.ctypes.data, 48, q_t.ctypes.data, 32, s.ctypes.data, 3)
    assert rc == 0
    return q_rm, q_t, s


def test_multi_tensor_call_equals_one_call_per_tensor():
    # several tensors in one call (mixed sizes, ragged edges, an empty one, an unaligned view): the bytes are those
    # of fp4q_quantize2d called once per tensor, hence the oracle's
    g = torch.Generator(device="cuda").manual_seed(12)
    shapes = [(256, 256), (100, 200), (0, 64), (384, 1024), (1, 1), (130, 72), (512, 128)]
    xs = [torch.randn(r, c, generator=g, device="cuda").to(torch.bfloat16) for r, c in shapes]
    big = torch.randn(260, 300, generator=g, device="cuda").to(torch.bfloat16)
    xs.append(big[3:200, 5:133])                                  # odd offset, pitch 300
    for mode in MODES:
        ids = [7 + 3 * j for j in range(len(xs))]
        outs = binding.fp4q_quantize2d_multi(xs, mode=mode, seed=21, tensor_ids=ids)
        torch.cuda.synchronize()
        for x, q, tid in zip(xs, outs, ids):
            if x.numel() == 0:
                continue
            one = gpu_quantize(x, mode, seed=21, tensor_id=tid)
            assert all(np.array_equal(a, b) for a, b in zip(logical(q), logical(one)))
        # and directly against the oracle for two of them
        for j in (1, 5):
            o_rm, o_t, o_s = oracle.quantize2d(workloads.bf16_bits(xs[j]), mode, 21, ids[j])
            g_rm, g_t, g_s = logical(outs[j])
            r, c = shapes[j]
            assert np.array_equal(g_s, o_s) and np.array_equal(g_rm[:, :(c + 1) // 2], o_rm) and np.array_equal(g_t[:, :(r + 1) // 2], o_t)


def test_multi_tensor_call_with_many_tensors():
    g = torch.Generator(device="cuda").manual_seed(13)
    xs = [torch.randn(64 + 32 * (j % 3), 96, generator=g, device="cuda").to(torch.bfloat16) for j in range(70)]
    outs = binding.fp4q_quantize2d_multi(xs, mode=binding.ROUND_STOCHASTIC, seed=5)
    torch.cuda.synchronize()
    for j in (0, 31, 32, 33, 69):
        one = gpu_quantize(xs[j], binding.ROUND_STOCHASTIC, seed=5, tensor_id=j)
        assert all(np.array_equal(a, b) for a, b in zip(logical(outs[j]), logical(one)))


def test_ragged_outputs_do_not_write_outside_their_extent():
    # the quantizers use plain stores: guard bytes before and after every output buffer must survive
    for rows, cols in [(33, 31), (100, 200), (129, 257), (1, 1)]:
        x = torch.randn(rows, cols, device="cuda").to(torch.bfloat16)
        q = binding.alloc_qtensor(rows, cols, "cuda")
        guard = 256
        bufs = {}
        for name in ("q_rm", "q_t", "scale"):
            t = getattr(q, name)
            flat = torch.full((guard + t.numel() + guard,), 0xA5, dtype=torch.uint8, device="cuda")
            bufs[name] = flat
            setattr(q, name, flat[guard:guard + t.numel()].view(t.shape))
        binding.fp4q_quantize2d(x, out=q, mode=binding.ROUND_STOCHASTIC, seed=3, tensor_id=1)
        torch.cuda.synchronize()
        for name, flat in bufs.items():
            assert bool((flat[:guard] == 0xA5).all()) and bool((flat[-guard:] == 0xA5).all()), (name, rows, cols)
        o_rm, o_t, o_s = oracle.quantize2d(workloads.bf16_bits(x), oracle.MODE_STOCHASTIC, 3, 1)
        assert np.array_equal(q.scale.cpu().numpy()[:, :o_s.shape[1]], o_s)
        assert np.array_equal(q.q_rm.cpu().numpy()[:, :o_rm.shape[1]], o_rm) and np.array_equal(q.q_t.cpu().numpy()[:, :o_t.shape[1]], o_t)
