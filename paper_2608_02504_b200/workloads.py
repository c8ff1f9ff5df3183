"""Seeded synthetic inputs shaped like the paper's video-DiT attention workloads.

This module only draws inputs; it holds none of the method's arithmetic and is the
one module both the CUDA path's callers and the CPU oracle's callers may share.

Recipe (per head, per token at raster index n = (t*H + y)*W + x):
    q = s * (u + P(t, y, x)),   k = u' + P(t, y, x),   v ~ N(0, 1)
with u, u' ~ N(0, 1)^d, s log-uniform in [s_lo, s_hi] (so query entropy spreads from
near 0 to near log N) and P a fixed three-axis sinusoidal embedding scaled by 2, which
makes <P(i), P(j)> peak at zero offset (query-centred neighbourhoods).  Everything is
rounded to bf16.  The tensors are returned in RASTER token order, [1, heads, N, d].

The real models' weights and prompt sets are not available, so these tensors stand in
for the Wan2.1 / Wan2.2 / HunyuanVideo attention inputs of the paper's experiments.
"""
from __future__ import annotations

import math

import numpy as np
import torch

CONFIGS = {
    # name: latent grid, heads, head_dim, block size, tile shape, query-scale range, decay, seed
    "tiny": dict(T=4, H=8, W=8, heads=2, head_dim=64, block=64, tile_h=4, tile_w=4,
                 s_lo=0.3, s_hi=3.0, gamma=0.6, tau=0.9, seed=1235),
    "wan1.3b-480p": dict(T=21, H=30, W=52, heads=12, head_dim=128, block=128, tile_h=8, tile_w=16,
                         s_lo=0.3, s_hi=3.0, gamma=0.6, tau=0.9, seed=1236),
    "wan14b-720p": dict(T=21, H=45, W=80, heads=40, head_dim=128, block=128, tile_h=8, tile_w=16,
                        s_lo=0.2, s_hi=5.0, gamma=0.6, tau=0.9, seed=1237),
    "hunyuan-720p": dict(T=33, H=45, W=80, heads=24, head_dim=128, block=128, tile_h=8, tile_w=16,
                         s_lo=0.3, s_hi=3.0, gamma=0.95, tau=0.9, seed=1238),
}


def num_tokens(cfg) -> int:
    return cfg["T"] * cfg["H"] * cfg["W"]


def _axis_embedding(pos: torch.Tensor, width: int) -> torch.Tensor:
    """[n] integer positions -> [n, width]; channel 2k = 2 sin(w_k p), 2k+1 = 2 cos(w_k p)."""
    k = torch.arange(width // 2, device=pos.device, dtype=torch.float32)
    omega = torch.pow(torch.tensor(10000.0, device=pos.device), -2.0 * k / float(width))
    ang = pos.to(torch.float32)[:, None] * omega[None, :]
    out = torch.empty(pos.numel(), width, device=pos.device, dtype=torch.float32)
    out[:, 0::2] = 2.0 * torch.sin(ang)
    out[:, 1::2] = 2.0 * torch.cos(ang)
    return out


def position_embedding(T: int, H: int, W: int, d: int, device) -> torch.Tensor:
    """P for every raster token: [T*H*W, d] fp32; d split as (d_t, d_h, d_w), d_h = d_w = 2*(d//6)."""
    d_h = d_w = 2 * (d // 6)
    d_t = d - d_h - d_w
    n = torch.arange(T * H * W, device=device)
    t = n // (H * W)
    y = (n // W) % H
    x = n % W
    return torch.cat([_axis_embedding(t, d_t), _axis_embedding(y, d_h), _axis_embedding(x, d_w)], dim=1)


def make_head_state(cfg, head: int, device="cpu"):
    """fp32 pre-rounding (q, k, v) of one head, each [N, d], raster order."""
    N, d = num_tokens(cfg), cfg["head_dim"]
    g = torch.Generator(device=device)
    g.manual_seed(cfg["seed"] * 1000003 + head)
    P = position_embedding(cfg["T"], cfg["H"], cfg["W"], d, device)
    u = torch.randn(N, d, generator=g, device=device)
    u2 = torch.randn(N, d, generator=g, device=device)
    v = torch.randn(N, d, generator=g, device=device)
    r = torch.rand(N, generator=g, device=device)
    s = torch.exp(math.log(cfg["s_lo"]) + r * (math.log(cfg["s_hi"]) - math.log(cfg["s_lo"])))
    q = s[:, None] * (u + P)
    k = u2 + P
    return q, k, v


def make_qkv(cfg, device="cpu", heads=None):
    """bf16 Q, K, V of shape [1, n_heads, N, d] in raster token order.

    ``heads`` selects a subset (list of head indices); each head has its own seed, so a
    subset reproduces the same values those heads have in the full tensor.
    """
    heads = list(range(cfg["heads"])) if heads is None else list(heads)
    N, d = num_tokens(cfg), cfg["head_dim"]
    Q = torch.empty(1, len(heads), N, d, dtype=torch.bfloat16, device=device)
    K = torch.empty_like(Q)
    V = torch.empty_like(Q)
    for i, h in enumerate(heads):
        q, k, v = make_head_state(cfg, h, device)
        Q[0, i] = q.to(torch.bfloat16)
        K[0, i] = k.to(torch.bfloat16)
        V[0, i] = v.to(torch.bfloat16)
    return Q, K, V


def append_text(Q, K, V, cfg, n_text: int, heads=None):
    """Joint text-video sequences: n_text text tokens after the video tokens of every head.
    Text tokens carry no position embedding: q = s * u, k = u', v ~ N(0, 1), from a generator of
    their own, so the video part is the tensor make_qkv returns.  Returns new [1, heads, N + n_text, d]."""
    heads = list(range(cfg["heads"])) if heads is None else list(heads)
    d, device = cfg["head_dim"], Q.device
    out = [torch.empty(1, len(heads), Q.shape[2] + n_text, d, dtype=torch.bfloat16, device=device) for _ in range(3)]
    for src, dst in zip((Q, K, V), out):
        dst[:, :, : Q.shape[2]] = src
    for i, h in enumerate(heads):
        g = torch.Generator(device=device)
        g.manual_seed(cfg["seed"] * 1000003 + 500000 + h)
        u = torch.randn(n_text, d, generator=g, device=device)
        u2 = torch.randn(n_text, d, generator=g, device=device)
        v = torch.randn(n_text, d, generator=g, device=device)
        r = torch.rand(n_text, generator=g, device=device)
        s = torch.exp(math.log(cfg["s_lo"]) + r * (math.log(cfg["s_hi"]) - math.log(cfg["s_lo"])))
        out[0][0, i, Q.shape[2]:] = (s[:, None] * u).to(torch.bfloat16)
        out[1][0, i, Q.shape[2]:] = u2.to(torch.bfloat16)
        out[2][0, i, Q.shape[2]:] = v.to(torch.bfloat16)
    return tuple(out)


def drift_(x: torch.Tensor, step: int, seed: int, sigma: float = 0.05) -> torch.Tensor:
    """Denoising-schedule emulation: x_t = x_{t-1} + sigma * N(0, 1), in place on an fp32 state."""
    g = torch.Generator(device=x.device)
    g.manual_seed(seed * 7919 + step)
    x.add_(torch.randn(x.shape, generator=g, device=x.device, dtype=x.dtype), alpha=sigma)
    return x


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
