"""Seeded random tensors (CPU, torch.Generator).  Draws only; no method arithmetic.

bf16 workloads are drawn in fp32 and rounded to bf16 once; both the oracle (which
widens them back to fp32) and the CUDA path consume those rounded values, so
parity measures kernel error rather than input quantisation.
"""
from __future__ import annotations

import numpy as np
import torch

from .configs import Config
from .layout import Layout

_CHUNK = 1 << 26  # elements per randn call (bounds the fp32 temporary)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def _torch_dtype(dtype: str):
    return torch.float32 if dtype == "f32" else torch.bfloat16


def _randn(shape, std: float, mean: float, dtype: str, g: torch.Generator, pin: bool = False):
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=_torch_dtype(dtype), pin_memory=pin)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        t = torch.randn(hi - lo, generator=g, dtype=torch.float32)
        if std != 1.0:
            t.mul_(std)
        if mean != 0.0:
            t.add_(mean)
        out[lo:hi] = t.to(out.dtype)
    return out.view(*shape)


def bf16_round(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16).to(torch.float32)


def draw_qkv(cfg: Config, lay: Layout, seed: int | None = None, std: float | None = None,
             pin: bool = False):
    """Q [T,H,D], K [T,Hkv,D], V [T,Hkv,D] ~ N(0, std)."""
    g = _gen((cfg.seed if seed is None else seed) * 7 + 1)
    s = cfg.qkv_std if std is None else std
    T = lay.total_tokens
    q = _randn((T, cfg.n_heads, cfg.head_dim), s, 0.0, cfg.dtype, g, pin)
    k = _randn((T, cfg.n_kv_heads, cfg.head_dim), s, 0.0, cfg.dtype, g, pin)
    v = _randn((T, cfg.n_kv_heads, cfg.head_dim), s, 0.0, cfg.dtype, g, pin)
    return q, k, v


def draw_logits(cfg: Config, lay: Layout, seed: int | None = None, pin: bool = False):
    """Logits [R, V] ~ N(0, logit_std); R = sum of query lengths, path-major."""
    g = _gen((cfg.seed if seed is None else seed) * 7 + 2)
    R = int(lay.qry_len.sum())
    return _randn((R, cfg.vocab), cfg.logit_std, 0.0, cfg.dtype, g, pin)


def draw_targets(cfg: Config, lay: Layout, seed: int | None = None) -> np.ndarray:
    """int32 [R]: uniform token ids; the last row of each path's block is -1
    (no next token to predict inside the segment)."""
    rng = np.random.default_rng((cfg.seed if seed is None else seed) * 7 + 3)
    R = int(lay.qry_len.sum())
    tgt = rng.integers(0, cfg.vocab, size=R).astype(np.int32)
    off = lay.query_row_offsets()
    tgt[off[1:][lay.qry_len > 0] - 1] = -1
    return tgt


def draw_prior_weight(cfg: Config, lay: Layout, seed: int | None = None):
    """prior_i ~ N(-2.5, 0.25) (a per-token document log-likelihood density);
    weight_i = 1 / query length."""
    rng = np.random.default_rng((cfg.seed if seed is None else seed) * 7 + 4)
    prior = rng.normal(-2.5, 0.25, size=lay.n_paths).astype(np.float32)
    weight = (1.0 / np.maximum(lay.qry_len, 1)).astype(np.float32)
    return prior, weight


def draw_decode_inputs(cfg: Config, n_prompts: int, steps: int, seed: int | None = None,
                       pin: bool = False):
    """Per-step decode inputs, before any position encoding:
    q [steps, B, H, D]; tail K, V [B, steps, Hkv, D] (row t is appended at step t)."""
    g = _gen((cfg.seed if seed is None else seed) * 7 + 5)
    q = _randn((steps, n_prompts, cfg.n_heads, cfg.head_dim), cfg.qkv_std, 0.0, cfg.dtype, g, pin)
    tk = _randn((n_prompts, steps, cfg.n_kv_heads, cfg.head_dim), cfg.qkv_std, 0.0, cfg.dtype, g, pin)
    tv = _randn((n_prompts, steps, cfg.n_kv_heads, cfg.head_dim), cfg.qkv_std, 0.0, cfg.dtype, g, pin)
    return q, tk, tv


def to_f32_numpy(t: torch.Tensor) -> np.ndarray:
    """Widen (exactly) to a contiguous float32 numpy array."""
    return t.detach().to("cpu").to(torch.float32).contiguous().numpy()
