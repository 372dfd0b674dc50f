"""Seeded synthetic inputs shaped like the paper's dense and MoE workloads.

This module holds no quantization or GEMM arithmetic: it only draws BF16 tensors
with the value distributions of the benchmark configurations and describes the
shapes of the linear layers.  Both the CUDA path and the CPU oracle consume the
bytes produced here.  The tensors stand in for weights, activations and
output-gradients of OLMo-1B/7B-class dense layers and a Qwen-30B-class MoE
expert layer (Section 4.1 lists the models); the real training tensors are not
available, so the distributions are synthetic: Gaussian weights, heavy-tailed
activations with a few outlier channels, and gradients with a log-normal
per-row scale.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Tuple

import numpy as np
import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def weights(rows: int, cols: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    """W ~ N(0, std^2), BF16."""
    g = _gen(seed, device)
    return (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def activations_gauss_outliers(rows: int, cols: int, seed: int, device="cpu", n_outlier_cols: int = 2,
                               outlier_scale: float = 50.0) -> torch.Tensor:
    """X ~ N(0,1) with a few seeded-random columns multiplied by outlier_scale."""
    g = _gen(seed, device)
    x = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    perm = torch.randperm(cols, generator=g, device=device)[:n_outlier_cols]
    x[:, perm] *= outlier_scale
    return x.to(torch.bfloat16)


def activations_student_t(rows: int, cols: int, seed: int, device="cpu", nu: int = 4,
                          outlier_frac: float = 0.005, outlier_scale: float = 30.0) -> torch.Tensor:
    """X ~ Student-t(nu) with a fraction of channels (columns) multiplied by outlier_scale."""
    g = _gen(seed, device)
    z = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    chi2 = torch.zeros(rows, cols, device=device, dtype=torch.float32)
    for _ in range(nu):
        chi2 += torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) ** 2
    x = z / torch.sqrt(chi2 / nu)
    del z, chi2
    n_out = int(round(outlier_frac * cols))
    if n_out > 0:
        perm = torch.randperm(cols, generator=g, device=device)[:n_out]
        x[:, perm] *= outlier_scale
    return x.to(torch.bfloat16)


def gradients_rowscaled(rows: int, cols: int, seed: int, device="cpu", sigma: float = 2.0) -> torch.Tensor:
    """dY ~ N(0,1) times a per-row log-normal(0, sigma) scale."""
    g = _gen(seed, device)
    y = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    s = torch.exp(torch.randn(rows, 1, generator=g, device=device, dtype=torch.float32) * sigma)
    return (y * s).to(torch.bfloat16)


def gradients_gauss(rows: int, cols: int, seed: int, device="cpu", std: float = 1e-3) -> torch.Tensor:
    g = _gen(seed, device)
    return (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The BF16 bit patterns of a tensor as a uint16 numpy array (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(bits: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


# ---------------------------------------------------------------------------------------------------
# Layer shapes.  A linear layer is (name, N = output features, K = input features); with T tokens the
# forward product is [T,K] x [N,K]^T, dgrad [T,N] x [N,K], wgrad [T,N]^T x [T,K].

@dataclass(frozen=True)
class DenseConfig:
    name: str
    tokens: int
    hidden: int
    ffn: int
    nu: int = 4
    data_seed: int = 0
    philox_seed: int = 0

    def layers(self) -> List[Tuple[str, int, int]]:
        h, f = self.hidden, self.ffn
        return [("q", h, h), ("k", h, h), ("v", h, h), ("o", h, h),
                ("gate", f, h), ("up", f, h), ("down", h, f)]

    def fwd_flops(self) -> float:
        return sum(2.0 * self.tokens * n * k for _, n, k in self.layers())


CONFIG_TINY = DenseConfig("tiny-linear-256", tokens=128, hidden=256, ffn=256, data_seed=100, philox_seed=0)
CONFIG_1B = DenseConfig("dense-1B-class", tokens=8192, hidden=2048, ffn=5632, data_seed=200, philox_seed=2)
CONFIG_7B = DenseConfig("dense-7B-class", tokens=16384, hidden=4096, ffn=11008, data_seed=300, philox_seed=3)
CONFIG_ATTN_7B = DenseConfig("attn-7B-mxfp8-qk", tokens=16384, hidden=4096, ffn=11008, nu=3, data_seed=400,
                             philox_seed=4)


def tiny_layer(device="cpu") -> Dict[str, torch.Tensor]:
    """The tiny linear layer: W 256x256 ~N(0,0.02), X 128x256 ~N(0,1) with 2 outlier columns x50,
    dY 128x256 ~N(0,1e-3)."""
    return {
        "W": weights(256, 256, 100, device),
        "X": activations_gauss_outliers(128, 256, 101, device),
        "dY": gradients_gauss(128, 256, 102, device),
    }


def dense_layer_tensors(cfg: DenseConfig, layer: Tuple[str, int, int], index: int, device="cpu",
                        tokens: int | None = None) -> Dict[str, torch.Tensor]:
    """W [N,K], X [T,K], dY [T,N] of one linear layer of a dense configuration."""
    _, n, k = layer
    t = cfg.tokens if tokens is None else tokens
    base = cfg.data_seed + 10 * index
    return {
        "W": weights(n, k, base, device),
        "X": activations_student_t(t, k, base + 1, device, nu=cfg.nu),
        "dY": gradients_rowscaled(t, n, base + 2, device),
    }


@dataclass(frozen=True)
class MoEConfig:
    name: str = "moe-30B-class-expert-layer"
    experts: int = 128
    hidden: int = 2048
    expert_ffn: int = 768
    tokens: int = 16384
    top_k: int = 8
    zipf: float = 1.2
    pad: int = 128
    data_seed: int = 500
    philox_seed: int = 5

    def layers(self) -> List[Tuple[str, int, int]]:
        return [("gate", self.expert_ffn, self.hidden), ("up", self.expert_ffn, self.hidden),
                ("down", self.hidden, self.expert_ffn)]


CONFIG_MOE = MoEConfig()


def moe_routing(cfg: MoEConfig, tokens: int | None = None, experts: int | None = None) -> np.ndarray:
    """Per-expert token counts: every token picks top_k distinct experts with p proportional to
    rank^-zipf (Gumbel-top-k sampling without replacement). Returns counts [E] (int64)."""
    t = cfg.tokens if tokens is None else tokens
    e = cfg.experts if experts is None else experts
    g = _gen(cfg.data_seed, "cpu")
    logp = -cfg.zipf * torch.log(torch.arange(1, e + 1, dtype=torch.float64))
    u = torch.rand(t, e, generator=g, dtype=torch.float64).clamp_(1e-300, 1.0)
    gumbel = -torch.log(-torch.log(u))
    top = torch.topk(logp[None, :] + gumbel, min(cfg.top_k, e), dim=1).indices
    return torch.bincount(top.reshape(-1), minlength=e).numpy().astype(np.int64)


def padded_row_offsets(counts: np.ndarray, pad: int = 128) -> np.ndarray:
    """Exclusive prefix sum of the group sizes rounded up to a multiple of pad: row_offsets[E+1]."""
    padded = (np.asarray(counts, dtype=np.int64) + pad - 1) // pad * pad
    return np.concatenate([[0], np.cumsum(padded)]).astype(np.int64)


def zero_padding_rows(t: torch.Tensor, counts: np.ndarray, row_offsets: np.ndarray) -> torch.Tensor:
    """Zero the rows of a permuted token matrix that lie between a group's valid rows and its padded end."""
    for g, c in enumerate(counts):
        t[int(row_offsets[g]) + int(c):int(row_offsets[g + 1])] = 0
    return t
