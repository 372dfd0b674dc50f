"""Straight-through FP4 linear layer on top of the C-ABI calls (glue only; every step runs in the library's kernels).

Section 3.1 of the paper: the forward product uses 2D-block-quantized weights and activations (round to nearest),
the backward pass quantizes the incoming gradient once (stochastic rounding) and uses it, with the quantized
operands saved by the forward pass, in both backward products; the quantizers are treated as identity when
differentiating (straight-through estimator).  Because the blocks are 32x32, the transposed payloads the backward
products need are written by the same quantization call: nothing is re-quantized between forward and backward.
"""
from __future__ import annotations

import torch

from . import binding


class _FP4LinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, weight, seed, tensor_id, ws):
        # x [T, K], weight [N, K]; both are quantized once, with both payload layouts
        qx = binding.fp4q_quantize2d(x.to(torch.bfloat16).contiguous(), mode=binding.ROUND_NEAREST)
        qw = binding.fp4q_quantize2d(weight.to(torch.bfloat16).contiguous(), mode=binding.ROUND_NEAREST)
        y = binding.fp4q_gemm_fwd(qx, qw, dt=binding.OUT_BF16, ws=ws)
        ctx.qx, ctx.qw, ctx.ws = qx, qw, ws
        ctx.seed, ctx.tensor_id = int(seed), int(tensor_id)
        ctx.x_dtype, ctx.w_dtype = x.dtype, weight.dtype
        return y if y.is_contiguous() else y.contiguous()

    @staticmethod
    def backward(ctx, dy):
        qdy = binding.fp4q_quantize2d(dy.to(torch.bfloat16).contiguous(), mode=binding.ROUND_STOCHASTIC,
                                      seed=ctx.seed, tensor_id=ctx.tensor_id)
        dx = dw = None
        if ctx.needs_input_grad[0]:
            dx = binding.fp4q_gemm_dgrad(qdy, ctx.qw, dt=binding.OUT_BF16, ws=ctx.ws).to(ctx.x_dtype)
        if ctx.needs_input_grad[1]:
            dw = binding.fp4q_gemm_wgrad(qdy, ctx.qx, dt=binding.OUT_F32, ws=ctx.ws).to(ctx.w_dtype)
        ctx.qx = ctx.qw = None
        return dx, dw, None, None, None


def fp4_linear(x: torch.Tensor, weight: torch.Tensor, seed: int = 0, tensor_id: int = 0, ws=None) -> torch.Tensor:
    """y = x^ weight^^T with FP4 forward and backward products.  x [..., K] and weight [N, K] live on the GPU;
    `seed` / `tensor_id` key the stochastic rounding of the incoming gradient (change one of them every step)."""
    if ws is None:
        ws = binding.alloc_workspace(x.device)
    lead = x.shape[:-1]
    y = _FP4LinearFn.apply(x.reshape(-1, x.shape[-1]), weight, seed, tensor_id, ws)
    return y.reshape(*lead, weight.shape[0])


class FP4Linear(torch.nn.Module):
    """Bias-free linear layer with an FP32 master weight and FP4 products.  Each backward pass draws fresh
    stochastic-rounding bits: the module counts its forward calls and uses the count as the Philox tensor id's
    high part, `layer_id` as the low 8 bits."""

    def __init__(self, in_features: int, out_features: int, layer_id: int = 0, seed: int = 0, device="cuda"):
        super().__init__()
        self.weight = torch.nn.Parameter(torch.empty(out_features, in_features, device=device, dtype=torch.float32))
        torch.nn.init.normal_(self.weight, std=0.02)
        self.layer_id, self.seed, self.calls = int(layer_id) & 0xFF, int(seed), 0
        self._ws = None

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        if self._ws is None or self._ws.device != x.device:
            self._ws = binding.alloc_workspace(x.device)
        self.calls += 1
        tid = ((self.calls & 0xFFFFFF) << 8) | self.layer_id
        return fp4_linear(x, self.weight, seed=self.seed, tensor_id=tid, ws=self._ws)
