"""Seeded synthetic KV caches shaped like the paper's models.

This module only manufactures inputs (window queries, cached keys and values)
for the tests and the benchmark.  It holds none of the Expected Attention
arithmetic and is the one module that both the CUDA path's tests and the CPU
oracle's tests may share.  torch is used for random numbers and bf16 rounding;
the same bits are handed to both sides.

Recipe, per layer (one ``torch.Generator`` seeded ``1000 * cfg_id + layer``):
  * an outlier channel set O (uniform, without replacement); ``scale_c`` is the
    outlier scale on O and 1 elsewhere; O is shared by every Q and K head;
  * per KV head: channel offsets ``off_k ~ N(0, 0.5^2)``, pre-RoPE keys
    ``bf16((z + off_k) * scale)``, then rotary embedding at the key's position
    (half-split pairing, ``theta_m = base^(-2m/d)``) and rounding to bf16;
    optionally the offsets drift along the sequence as a random walk;
  * per query head: offsets ``off_q ~ N(0, 0.5^2)``, a rank-rho mixing factor
    ``F ~ N(0,1)/sqrt(rho)``; window queries ``bf16((z + yF + off_q) * scale)``
    with ``y ~ N(0, I_rho)``; queries stay pre-RoPE;
  * per KV head: values ``bf16(z * exp(0.5 g_i))`` with one ``g_i ~ N(0,1)`` per
    token (log-normal token scale).
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class EAConfig:
    name: str
    cfg_id: int
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_keys: int
    window: int
    n_future: int
    rope_base: float
    n_kept: int
    n_outliers: int
    outlier_scale: float
    q_rank: int
    drift_sigma: float = 0.0
    eps: float = 0.02

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_units(self) -> int:
        return self.n_layers * self.batch

    @property
    def key_slots(self) -> int:
        return self.n_units * self.n_kv_heads * self.n_keys

    def tempered(self, outlier_scale: float, eps: float | None = None) -> "EAConfig":
        """Same shapes with milder outliers: the softmax is then spread over many keys."""
        return dataclasses.replace(
            self, name=f"{self.name}-x{outlier_scale:g}" + ("" if eps is None else f"-eps{eps:g}"),
            outlier_scale=outlier_scale, eps=self.eps if eps is None else eps)


CONFIGS = {
    # tiny single layer
    0: EAConfig("cfg0-tiny", 0, 1, 1, 4, 2, 64, 512, 64, 512, 1e4, 256, 2, 20.0, 8),
    # Llama3.1-8B-shaped single layer
    1: EAConfig("cfg1-llama8b-layer", 1, 1, 1, 32, 8, 128, 8192, 128, 512, 5e5, 4096, 4, 30.0, 16),
    # Qwen3-8B-shaped full stack
    2: EAConfig("cfg2-qwen3-8b-32k", 2, 36, 1, 32, 8, 128, 32768, 128, 512, 1e6, 8192, 4, 30.0, 16),
    # Gemma3-12B-shaped 128k context
    3: EAConfig("cfg3-gemma3-12b-128k", 3, 48, 1, 16, 8, 256, 131072, 256, 1024, 1e6, 16384, 2,
                20.0, 8, drift_sigma=0.01),
    # decode-phase streaming (one compression event; see decode_schedule)
    4: EAConfig("cfg4-qwen7b-r1-decode", 4, 28, 8, 28, 4, 128, 4608, 128, 512, 1e6, 4096, 2, 20.0,
                8),
}


def decode_schedule(start: int = 2048, end: int = 16384, every: int = 512, budget: int = 4096):
    """Compression events of the streaming config: (absolute position, keys in cache, kept)."""
    events, cache, pos = [], start, start
    while pos < end:
        pos += every
        n = cache + every
        kept = min(n, budget)
        events.append((pos, n, kept))
        cache = kept
    return events


def rope_half_split(x: torch.Tensor, positions: torch.Tensor, rope_base: float) -> torch.Tensor:
    """Rotary embedding of fp32 rows ``x[..., n, d]`` at integer ``positions[n]``.

    Channel m is paired with m + d/2; angle = position * base^(-2m/d).
    """
    d = x.shape[-1]
    half = d // 2
    m = torch.arange(half, device=x.device, dtype=torch.float64)
    theta = torch.pow(torch.tensor(rope_base, dtype=torch.float64, device=x.device), -2.0 * m / d)
    ang = positions.to(torch.float64)[:, None] * theta[None, :]
    cos, sin = torch.cos(ang).float(), torch.sin(ang).float()
    a, b = x[..., :half], x[..., half:]
    return torch.cat([a * cos - b * sin, a * sin + b * cos], dim=-1)


def generate_layer(cfg: EAConfig, layer: int = 0, device="cpu", n_keys: int | None = None,
                   key_positions: torch.Tensor | None = None, pos_next: int | None = None,
                   q_phase: float | None = None, draw: int = 0):
    """One layer of synthetic activations.

    Returns ``(q_win [B,Hq,W,d], k [B,Hkv,n,d], v [B,Hkv,n,d], pos_next [B] int64)``; the three
    tensors are bf16 on ``device``.  ``q_phase`` (streaming config) rotates the query offsets
    between two fixed directions: ``off_q = cos(phase) A + sin(phase) B``.  ``draw`` > 0 gives further
    independent draws of the noise with the layer's outlier channels, offsets and query factor unchanged
    (the tokens generated between two compression events of a stream).
    """
    n = cfg.n_keys if n_keys is None else n_keys
    B, Hq, Hkv, d, W = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1000 * cfg.cfg_id + layer)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32)

    perm = torch.randperm(d, generator=gen, device=dev)
    scale = torch.ones(d, device=dev)
    scale[perm[: cfg.n_outliers]] = cfg.outlier_scale

    # what belongs to the layer (drawn first, from the layer's seed): channel offsets and the query factor
    off_k = 0.5 * randn(B, Hkv, 1, d)
    if draw:
        off_a = 0.5 * randn(B, Hq, 1, d)
        off_b = 0.5 * randn(B, Hq, 1, d)
        F = randn(B, Hq, cfg.q_rank, d) / math.sqrt(cfg.q_rank)
        gen.manual_seed(1000 * cfg.cfg_id + layer + 7919 * draw)      # the noise of this draw

    # keys
    k_pre = randn(B, Hkv, n, d)
    if cfg.drift_sigma > 0:
        k_pre += torch.cumsum(cfg.drift_sigma * randn(B, Hkv, n, d), dim=2)
    k_pre = ((k_pre + off_k) * scale).to(torch.bfloat16).float()
    if key_positions is None:
        key_positions = torch.arange(n, device=dev)
    k = rope_half_split(k_pre, key_positions.to(dev), cfg.rope_base).to(torch.bfloat16)
    del k_pre

    # window queries (pre-RoPE)
    if not draw:
        off_a = 0.5 * randn(B, Hq, 1, d)
        off_b = 0.5 * randn(B, Hq, 1, d)
    off_q = off_a if q_phase is None else math.cos(q_phase) * off_a + math.sin(q_phase) * off_b
    if not draw:
        F = randn(B, Hq, cfg.q_rank, d) / math.sqrt(cfg.q_rank)
    y = randn(B, Hq, W, cfg.q_rank)
    q = ((randn(B, Hq, W, d) + y @ F + off_q) * scale).to(torch.bfloat16)

    # values
    g = randn(B, Hkv, n, 1)
    v = (randn(B, Hkv, n, d) * torch.exp(0.5 * g)).to(torch.bfloat16)

    p = n if pos_next is None else pos_next
    return q, k, v, torch.full((B,), p, dtype=torch.int64)


def quantize_e4m3(k: torch.Tensor, v: torch.Tensor, k_scale: torch.Tensor | None = None):
    """Manufactures a quantised cache from bf16 ``k, v`` [B,Hkv,n,d]: FP8 E4M3 codes (uint8) with one fp32
    scale per key channel and one per value token, each scale mapping the largest magnitude to 448.
    Returns ``(k_q8, k_scale [B,Hkv,d], v_q8, v_scale [B,Hkv,n])``.  Rounding is torch's cast.  With
    ``k_scale`` given (pairs appended to an existing cache) the keys are coded against those scales,
    saturating at the largest finite code."""
    kf, vf = k.float(), v.float()
    if k_scale is None:
        k_scale = (kf.abs().amax(dim=2) / 448.0).clamp_min(1e-30)
    v_scale = (vf.abs().amax(dim=3) / 448.0).clamp_min(1e-30)
    k_q8 = (kf / k_scale[:, :, None, :]).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
    v_q8 = (vf / v_scale[..., None]).to(torch.float8_e4m3fn).view(torch.uint8)
    return k_q8.contiguous(), k_scale.contiguous(), v_q8.contiguous(), v_scale.contiguous()


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array with the same bit patterns (host copy)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")
