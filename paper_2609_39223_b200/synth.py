"""Seeded synthetic inputs shaped like the paper's workloads.

This module serves both the CUDA path and the test oracle and therefore holds none of the
method's arithmetic: it only draws Gaussian tensors at the usual scales, plants outliers, and
routes tokens for the mixture-of-experts case. The paper trains real checkpoints on real text;
these tensors stand in for them (Gaussian weights at init scale, activation outlier channels).

All tensors are BF16 (rounded from FP32 by torch). The same bytes are handed to both sides.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def randn_bf16(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std^2) drawn in FP32 from a seeded generator on ``device``, rounded to BF16.
    Drawn in row chunks so that no FP32 copy of a large tensor is ever alive."""
    g = _gen(seed, device)
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for s in range(0, flat.numel(), step):
        n = min(step, flat.numel() - s)
        flat[s:s + n] = (torch.randn(n, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def weight_with_outliers(rows: int, cols: int, std: float = 0.02, frac: float = 1e-3, factor: float = 20.0,
                         seed: int = 0, device="cpu") -> torch.Tensor:
    """Weight matrix ~ N(0, std) with a seeded fraction of entries scaled by ``factor``."""
    w = randn_bf16((rows, cols), std, seed, device).float()
    g = _gen(seed + 1_000_003, device)
    n_out = int(round(rows * cols * frac))
    idx = torch.randperm(rows * cols, generator=g, device=device)[:n_out]
    w.view(-1)[idx] *= factor
    return w.to(torch.bfloat16)


def activations_with_outlier_channels(rows: int, cols: int, n_channels: int = 8, factor: float = 30.0,
                                      seed: int = 0, device="cpu") -> torch.Tensor:
    """Activations ~ N(0, 1) with ``n_channels`` seeded columns scaled by ``factor``."""
    x = randn_bf16((rows, cols), 1.0, seed, device)
    g = _gen(seed + 2_000_003, "cpu")
    ch = torch.randperm(cols, generator=g)[:n_channels].to(x.device)
    x[:, ch] = (x[:, ch].float() * factor).to(torch.bfloat16)
    return x


# ---- the five workload shapes ---------------------------------------------------------------

def nvfp4_weight_2048(device="cpu") -> torch.Tensor:
    """One 2048x2048 weight, N(0, 0.02), 0.1% of entries x20, seed 0."""
    return weight_with_outliers(2048, 2048, 0.02, 1e-3, 20.0, seed=0, device=device)


@dataclass
class LinearCase:
    X: torch.Tensor
    W: torch.Tensor
    dY: torch.Tensor


def linear_case(M: int, N: int, K: int, seed: int = 0, device="cpu", outlier_channels: int = 8,
                x_std: float = 1.0, w_std: float = 0.02, dy_std: float = 1e-3) -> LinearCase:
    """X [M,K] ~ N(0,1) with outlier channels x30, W [N,K] ~ N(0,0.02), dY [M,N] ~ N(0,1e-3)."""
    if outlier_channels:
        X = activations_with_outlier_channels(M, K, outlier_channels, 30.0, seed=seed, device=device)
        if x_std != 1.0:
            X = (X.float() * x_std).to(torch.bfloat16)
    else:
        X = randn_bf16((M, K), x_std, seed, device)
    W = randn_bf16((N, K), w_std, seed + 11, device)
    dY = randn_bf16((M, N), dy_std, seed + 23, device)
    return LinearCase(X, W, dY)


# 32-layer dense decoder: hidden 4096, MLP 14336 (SwiGLU), 32 query heads / 8 KV heads of dim 128.
DENSE_DECODER_LAYER = (
    ("q_proj", 4096, 4096), ("k_proj", 1024, 4096), ("v_proj", 1024, 4096), ("o_proj", 4096, 4096),
    ("gate_proj", 14336, 4096), ("up_proj", 14336, 4096), ("down_proj", 4096, 14336),
)
DENSE_DECODER_LAYERS = 32


def dense_decoder_layer_elems() -> int:
    return sum(r * c for _, r, c in DENSE_DECODER_LAYER)


def dense_decoder_weight(layer: int, name: str, device="cpu") -> torch.Tensor:
    for i, (n, r, c) in enumerate(DENSE_DECODER_LAYER):
        if n == name:
            return randn_bf16((r, c), 0.02, seed=layer * 16 + i, device=device)
    raise KeyError(name)


@dataclass
class MoeRouting:
    token_of_row: torch.Tensor     # [rows_padded] int64, -1 for padding rows
    group_offsets: torch.Tensor    # [G+1] int32, padded segment starts (multiples of ``align``)
    counts: torch.Tensor           # [G] int64, real rows per expert


def moe_routing(tokens: int, experts: int, top_k: int, seed: int = 0, align: int = 128) -> MoeRouting:
    """Top-k routing from the softmax of N(0,1) router logits (ties to the lower expert index),
    rows sorted by expert, each expert segment padded to a multiple of ``align`` rows."""
    g = _gen(seed, "cpu")
    logits = torch.randn(tokens, experts, generator=g, dtype=torch.float32)
    probs = torch.softmax(logits, dim=-1)
    # stable descending sort => ties resolved toward the lower index
    order = torch.sort(probs, dim=-1, descending=True, stable=True).indices[:, :top_k]
    expert = order.reshape(-1)
    token = torch.arange(tokens).repeat_interleave(top_k)
    perm = torch.sort(expert, stable=True).indices
    expert_sorted, token_sorted = expert[perm], token[perm]
    counts = torch.bincount(expert_sorted, minlength=experts)
    padded = (counts + align - 1) // align * align
    offs = torch.zeros(experts + 1, dtype=torch.int64)
    offs[1:] = torch.cumsum(padded, 0)
    token_of_row = torch.full((int(offs[-1]),), -1, dtype=torch.int64)
    start_real = torch.zeros(experts + 1, dtype=torch.int64)
    start_real[1:] = torch.cumsum(counts, 0)
    for e in range(experts):
        n = int(counts[e])
        token_of_row[int(offs[e]):int(offs[e]) + n] = token_sorted[int(start_real[e]):int(start_real[e]) + n]
    return MoeRouting(token_of_row, offs.to(torch.int32), counts)


def gather_rows(x: torch.Tensor, token_of_row: torch.Tensor) -> torch.Tensor:
    """Rows of ``x`` permuted into expert order; padding rows are zero."""
    out = torch.zeros((token_of_row.numel(), x.shape[1]), dtype=x.dtype, device=x.device)
    real = token_of_row >= 0
    out[real.to(x.device)] = x[token_of_row[real].to(x.device)]
    return out
