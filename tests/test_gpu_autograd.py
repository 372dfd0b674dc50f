"""GPU tests of the straight-through FP4 linear layer (Section 3.1): its three products against the oracle's, and a
dataset-free training smoke test (a student layer fits a random teacher)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2607_24953_b200 import autograd, workloads


def test_forward_and_backward_match_the_oracle_products():
    t = workloads.tiny_layer("cuda")
    x = t["X"].clone().requires_grad_(True)
    w = t["W"].clone().requires_grad_(True)
    dy = t["dY"]
    y = autograd.fp4_linear(x, w, seed=7, tensor_id=3)
    y.backward(dy)
    torch.cuda.synchronize()

    def dequantized(v, mode, **kw):
        bits = workloads.bf16_bits(v.cpu())
        q_rm, _, scale = oracle.quantize2d(bits, mode, **kw)
        return oracle.dequantize2d(q_rm, scale, bits.shape[0], bits.shape[1])

    xd = dequantized(t["X"], oracle.MODE_NEAREST)
    wd = dequantized(t["W"], oracle.MODE_NEAREST)
    dyd = dequantized(dy, oracle.MODE_STOCHASTIC, seed=7, tensor_id=3)
    for got, want, name in ((y, oracle.gemm_fwd(xd, wd), "forward"),
                            (x.grad, oracle.gemm_dgrad(dyd, wd), "dgrad"),
                            (w.grad, oracle.gemm_wgrad(dyd, xd), "wgrad")):
        got = got.detach().double().cpu().numpy()
        want = oracle.bf16_round(want)   # all three leave the layer in BF16
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert rel <= 1e-3, (name, rel)
        # and, per output row, max |G - O| <= 1e-2 * ||O_row||_inf
        assert (np.abs(got - want) <= 1e-2 * np.abs(want).max(axis=1, keepdims=True)).all(), name


def test_student_fits_a_random_teacher():
    torch.manual_seed(0)
    k, n, tokens = 256, 128, 512
    teacher = torch.randn(n, k, device="cuda") * 0.05
    student = autograd.FP4Linear(k, n, layer_id=1, seed=11)
    # mean-squared loss over tokens x outputs: the curvature is 2/n, so a step of n/8 contracts the error by 3/4
    opt = torch.optim.SGD(student.parameters(), lr=n / 8)
    losses = []
    for step in range(100):
        x = torch.randn(tokens, k, device="cuda", dtype=torch.bfloat16)
        target = (x.float() @ teacher.t())
        loss = ((student(x).float() - target) ** 2).mean()
        opt.zero_grad()
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    assert np.isfinite(losses).all()
    # down to the FP4 noise floor (the quantization error of the student's own forward product: a few percent)
    assert np.mean(losses[-10:]) < 0.05 * losses[0], (losses[0], losses[-10:])
