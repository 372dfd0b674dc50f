"""What the 8 random bits of the stochastic-rounding rule cost (reading R7 of the rounding appendix).

The paper asks for E[roundS(x)] = x (Section 3.1).  With 8 random bits an element between neighbours lo <= v < hi
goes up with probability floor(256 p) / 256, p = (v - lo) / (hi - lo): exactly unbiased when 256 p is an integer
(every BF16 v >= 0.25 after scaling), otherwise biased toward zero by less than (hi - lo) / 256.  In the weight
gradient dW = dY^T X that bias adds up linearly over the tokens while the rounding noise grows like the square
root of their number, so the question is whether the bias stays below the noise at the token counts of the
benchmark configurations.  This test computes both, exactly, from the rule's own probabilities on the 1B-class
gradient distribution (N(0,1) times a per-row log-normal(0, 2) scale) at 16384 tokens."""
import numpy as np

import oracle
from paper_2607_24953_b200 import workloads

GRID = np.array([oracle.e2m1_value(c) for c in range(8)])


def _rule_moments(v):
    """Mean and variance of the rounded magnitude of scaled magnitudes v in [0, 6] under the 8-bit rule."""
    lo_i = np.searchsorted(GRID, v, side="right") - 1
    hi_i = np.minimum(lo_i + 1, 7)
    lo, hi = GRID[lo_i], GRID[hi_i]
    step = np.where(hi > lo, hi - lo, 1.0)
    P = np.floor(256.0 * (v - lo) / step) / 256.0
    return lo + step * P, step * step * P * (1.0 - P)


def test_rule_moments_are_those_of_the_oracle():
    # the closed form above against the oracle's rounding function enumerated over all 256 random bytes
    rng = np.random.default_rng(0)
    vs = np.concatenate([rng.uniform(0, 6, 40), rng.uniform(0, 0.25, 40), GRID, [0.001, 0.2499, 5.999]])
    mean, var = _rule_moments(vs)
    for v, m, s2 in zip(vs, mean, var):
        out = np.array([oracle.e2m1_value(oracle.round_stochastic(float(v), r)) for r in range(256)])
        assert abs(out.mean() - m) < 1e-12 and abs(out.var() - s2) < 1e-12


def test_accumulated_bias_of_the_weight_gradient_stays_below_the_rounding_noise():
    T, N, K = 16384, 48, 48
    dy = workloads.gradients_rowscaled(T, N, 202, "cpu").double().numpy()
    x_bits = workloads.bf16_bits(workloads.activations_student_t(T, K, 201, "cpu"))
    q, _, s = oracle.quantize2d(x_bits, oracle.MODE_NEAREST, want_t=False)
    x_hat = oracle.dequantize2d(q, s, T, K)                               # the other operand as the product sees it
    # block scales of dY (32 x 32 blocks, truncation-free), from the oracle's own scale rule
    S = np.empty_like(dy)
    for I in range(T // 32):
        for J in range((N + 31) // 32):
            m = np.abs(dy[32 * I:32 * I + 32, 32 * J:32 * J + 32]).max()
            S[32 * I:32 * I + 32, 32 * J:32 * J + 32] = np.ldexp(1.0, oracle.scale_exponent(m))
    mean, var = _rule_moments(np.abs(dy) / S)
    bias_elem = np.sign(dy) * (mean * S - np.abs(dy))                     # E[dY^] - dY, toward zero
    var_elem = var * S * S
    bias_dw = bias_elem.T @ x_hat                                          # adds up linearly over the tokens
    noise_dw = np.sqrt(var_elem.T @ (x_hat * x_hat))                       # standard deviation of the rounding noise
    ratio = np.abs(bias_dw) / noise_dw
    # at 16384 tokens the systematic part is a small fraction of one standard deviation of the noise, everywhere
    assert ratio.max() < 0.05, ratio.max()
    assert np.median(ratio) < 0.01, np.median(ratio)
    # in Frobenius norm the systematic part is about a hundredth of the noise (the figures quoted in the design notes)
    frob = np.linalg.norm(bias_dw) / np.linalg.norm(noise_dw)
    assert frob < 0.02, frob
    print("bias / noise: max %.4f median %.4f Frobenius %.4f" % (ratio.max(), np.median(ratio), frob))
