"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors (torch generators, CPU or CUDA); it holds none of the method's arithmetic and
is the one module both the CUDA path's tests/benchmark and the CPU oracle's callers use.  The tensors stand in for the
training tensors of the paper's Dense-1.5B and MoE-7.9B / MoE-124B models (Sec. 5), which are not available: shapes
follow those layer classes, value distributions are heavy-tailed activations with a few outlier channels, small
Gaussian weights and tiny, per-token-scaled gradients.
"""
from __future__ import annotations

import math

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _chunks(rows: int, cols: int, max_elems: int = 1 << 26):
    step = max(1, max_elems // max(cols, 1))
    for r0 in range(0, rows, step):
        yield r0, min(rows, r0 + step)


def normal_bf16(rows: int, cols: int, std: float, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std²) entries, BF16 [rows][cols]."""
    g = _gen(seed, device)
    out = torch.empty(rows, cols, dtype=torch.bfloat16, device=device)
    for r0, r1 in _chunks(rows, cols):
        out[r0:r1] = (torch.randn(r1 - r0, cols, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def heavy_tailed_activations(rows: int, cols: int, seed: int, n_outlier_channels: int = 8, outlier_gain: float = 30.0,
                             device="cpu") -> torch.Tensor:
    """Student-t (nu = 3) entries with a few seeded channels (columns) multiplied by outlier_gain, BF16."""
    g = _gen(seed, device)
    gc = _gen(seed + 7919, "cpu")
    n_out = min(n_outlier_channels, cols)
    channels = torch.randperm(cols, generator=gc)[:n_out].to(device)
    out = torch.empty(rows, cols, dtype=torch.bfloat16, device=device)
    for r0, r1 in _chunks(rows, cols, 1 << 24):
        z = torch.randn(4, r1 - r0, cols, generator=g, device=device, dtype=torch.float32)
        t = z[0] / torch.sqrt((z[1] ** 2 + z[2] ** 2 + z[3] ** 2) / 3.0)
        t[:, channels] *= outlier_gain
        out[r0:r1] = t.to(torch.bfloat16)
    return out


def token_scaled_gradients(rows: int, cols: int, std: float, seed: int, sigma_log: float = 1.0,
                           device="cpu") -> torch.Tensor:
    """N(0, std²) entries times a log-normal per-row (per-token) factor exp(N(0, sigma_log²)), BF16."""
    g = _gen(seed, device)
    out = torch.empty(rows, cols, dtype=torch.bfloat16, device=device)
    for r0, r1 in _chunks(rows, cols):
        scale = torch.exp(torch.randn(r1 - r0, 1, generator=g, device=device, dtype=torch.float32) * sigma_log)
        out[r0:r1] = (torch.randn(r1 - r0, cols, generator=g, device=device, dtype=torch.float32) * std * scale).to(
            torch.bfloat16)
    return out


def spiky_normal(rows: int, cols: int, seed: int, spike_prob: float = 1e-3, spike_gain: float = 50.0,
                 device="cpu") -> torch.Tensor:
    """N(0,1) entries of which a seeded Bernoulli(spike_prob) subset is multiplied by spike_gain, BF16."""
    g = _gen(seed, device)
    out = torch.empty(rows, cols, dtype=torch.bfloat16, device=device)
    for r0, r1 in _chunks(rows, cols):
        x = torch.randn(r1 - r0, cols, generator=g, device=device, dtype=torch.float32)
        m = torch.rand(r1 - r0, cols, generator=g, device=device, dtype=torch.float32) < spike_prob
        out[r0:r1] = torch.where(m, x * spike_gain, x).to(torch.bfloat16)
    return out


def tiny_layer(seed: int = 0, device="cpu"):
    """The tiny single-layer check: X 256x256 ~ N(0,1), W 256x256 ~ N(0, 0.02²), dY 256x256 ~ N(0, (1e-3)²)."""
    return (normal_bf16(256, 256, 1.0, seed * 3 + 0, device),
            normal_bf16(256, 256, 0.02, seed * 3 + 1, device),
            normal_bf16(256, 256, 1e-3, seed * 3 + 2, device))


def dense_layer(tokens: int, in_features: int, out_features: int, seed: int, device="cpu"):
    """One dense linear layer of the Dense-1.5B class: X [T][in], W [out][in], dY [T][out]."""
    X = heavy_tailed_activations(tokens, in_features, seed * 3 + 0, device=device)
    W = normal_bf16(out_features, in_features, 0.02, seed * 3 + 1, device)
    dY = token_scaled_gradients(tokens, out_features, 1e-4, seed * 3 + 2, device=device)
    return X, W, dY


def moe_routing(n_experts: int, tokens: int, top_k: int, seed: int, zipf_s: float = 1.1, pad_to: int = 128):
    """Per-expert routed-row counts under a Zipf(s) expert popularity law with top-k routing.

    Every token draws top_k DISTINCT experts without replacement with weights (e+1)^-s (Gumbel top-k), so no expert
    can receive more than `tokens` rows.  Returns (counts[E], offsets[E+1]) as int64 CPU tensors; offsets are the
    prefix sums of the counts rounded up to a multiple of pad_to (padding rows are zero rows).
    """
    g = _gen(seed, "cpu")
    logw = -zipf_s * torch.log(torch.arange(1, n_experts + 1, dtype=torch.float64))
    counts = torch.zeros(n_experts, dtype=torch.int64)
    step = 1 << 14
    for t0 in range(0, tokens, step):
        n = min(step, tokens - t0)
        u = torch.rand(n, n_experts, generator=g, dtype=torch.float64).clamp_(1e-300, 1.0)
        gumbel = -torch.log(-torch.log(u))
        picks = torch.topk(logw + gumbel, top_k, dim=1).indices
        counts += torch.bincount(picks.reshape(-1), minlength=n_experts)
    padded = (counts + pad_to - 1) // pad_to * pad_to
    offsets = torch.zeros(n_experts + 1, dtype=torch.int64)
    offsets[1:] = torch.cumsum(padded, 0)
    return counts, offsets


def moe_layer(n_experts: int, hidden: int, ffn: int, tokens: int, top_k: int, seed: int, device="cpu"):
    """One MoE expert layer: X [rows][hidden] grouped by expert (padding rows zero), W [E*ffn][hidden],
    dY [rows][ffn], with counts/offsets from moe_routing."""
    counts, offsets = moe_routing(n_experts, tokens, top_k, seed * 5 + 3)
    rows = int(offsets[-1])
    X = heavy_tailed_activations(rows, hidden, seed * 5 + 0, device=device)
    dY = normal_bf16(rows, ffn, 1e-4, seed * 5 + 2, device)
    valid = torch.zeros(rows, dtype=torch.bool)
    for e in range(n_experts):
        valid[int(offsets[e]):int(offsets[e]) + int(counts[e])] = True
    valid = valid.to(device)
    X[~valid] = 0
    dY[~valid] = 0
    W = normal_bf16(n_experts * ffn, hidden, 0.02, seed * 5 + 1, device)
    return X, W, dY, counts, offsets


def bf16_bits(t: torch.Tensor):
    """Raw BF16 bit patterns of a tensor as a numpy uint16 array (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.uint16).numpy()
