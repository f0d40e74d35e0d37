"""Quantised-cache variant of the fp64 CPU oracle (8-bit keys and values with scales).

TEST INFRASTRUCTURE ONLY (see ``ea_oracle.py``).  The paper calls quantisation orthogonal to
eviction and combinable with it (Related Works, "Quantization" paragraph) and fixes no format; the
format taken here is a reading: keys and values stored as FP8 E4M3 codes (the OCP 8-bit
floating-point format: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, the
all-ones code is NaN, largest finite value 448), keys with one fp32 scale per (unit, KV head,
channel), values with one fp32 scale per (unit, KV head, token):

    k[u,g,i,c] = decode(k_q8[u,g,i,c]) * k_scale[u,g,c]
    v[u,g,i,c] = decode(v_q8[u,g,i,c]) * v_scale[u,g,i]

Scoring a quantised cache IS scoring the dequantised cache with the method's formulas (Eq. 7, 8, 9),
written out here in numpy fp64 with plain array expressions, no blocking or fusion.  Selection and
gathering are the integer routines of ``ea_oracle`` applied to codes and scales.

Parity status: pinned (``tests/test_oracle_pins.py``): the decoder against a library conversion of all
256 codes; dequantise-then-score against scoring with the key scales folded into the statistics (an
exact identity); unit scales and representable values against the pinned bf16 oracle; the ragged gather
of head-adaptive eviction against the pinned C routine on the same bytes and, where every head keeps
the same count, against plain indexing.
"""
from __future__ import annotations

import numpy as np

from oracle import ea_oracle


def e4m3_decode(codes) -> np.ndarray:
    """uint8 codes -> float64 values of FP8 E4M3 (finite-only variant; the NaN code decodes to nan)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    subnormal = (m / 8.0) * 2.0 ** -6
    val = np.where(e == 0, subnormal, normal)
    val = np.where((e == 15) & ((c & 0x7) == 7), np.nan, val)
    return sign * val


def dequant_k(k_q8, k_scale) -> np.ndarray:
    """k_q8 uint8 [U,Hkv,n,d], k_scale float [U,Hkv,d] -> float64 keys."""
    return e4m3_decode(k_q8) * np.asarray(k_scale, dtype=np.float64)[:, :, None, :]


def dequant_v(v_q8, v_scale) -> np.ndarray:
    """v_q8 uint8 [U,Hkv,n,d], v_scale float [U,Hkv,n] -> float64 values."""
    return e4m3_decode(v_q8) * np.asarray(v_scale, dtype=np.float64)[:, :, :, None]


def logits(k, mu_bar, sigma_bar) -> np.ndarray:
    """Eq. 7 on real-valued keys k [U,Hkv,n,d]: s[u,h,i] = mu_bar_h . k_i / sqrt(d) + k_i^T sigma_bar_h k_i / (2d)
    with query head h reading KV head h // G."""
    U, Hkv, n, d = k.shape
    Hq = mu_bar.shape[1]
    G = Hq // Hkv
    s = np.empty((U, Hq, n))
    for u in range(U):
        for h in range(Hq):
            kk = k[u, h // G]
            s[u, h] = kk @ mu_bar[u, h] / np.sqrt(d) + np.einsum("ia,ab,ib->i", kk, sigma_bar[u, h], kk) / (2 * d)
    return s


def scores(s, v, eps, group_mode=ea_oracle.GROUP_MEAN_PROB) -> np.ndarray:
    """Eq. 8 and Eq. 9 (with ||v||) on real-valued values v [U,Hkv,n,d]; the group modes of ``ea_oracle``."""
    U, Hq, n = s.shape
    Hkv = v.shape[1]
    G = Hq // Hkv
    vnorm = np.sqrt((v ** 2).sum(-1))

    def softmax(x):
        m = x.max(-1, keepdims=True)
        e = np.exp(x - m)
        return e / e.sum(-1, keepdims=True)

    if group_mode == ea_oracle.GROUP_MEAN_LOGIT:
        a = softmax(s.reshape(U, Hkv, G, n).mean(2))
    else:
        a = softmax(s).reshape(U, Hkv, G, n).sum(2)
        if group_mode == ea_oracle.GROUP_MEAN_PROB:
            a = a / G
    return (a + eps) * vnorm


def compress(q_win_bits, k_q8, k_scale, v_q8, v_scale, pos_next, n_future, rope_base, eps, n_kept,
             group_mode=ea_oracle.GROUP_MEAN_PROB):
    """Whole path on a quantised cache: statistics as ``ea_oracle.query_stats``, scores of the dequantised
    pairs, the eviction rule, and the kept codes with their scales (value scales follow their tokens, key
    scales belong to the channels and stay)."""
    mu_bar, sigma_bar = ea_oracle.query_stats(q_win_bits, np.asarray(pos_next, dtype=np.int64), n_future, rope_base)
    s = logits(dequant_k(k_q8, k_scale), mu_bar, sigma_bar)
    sc = scores(s, dequant_v(v_q8, v_scale), eps, group_mode)
    idx = ea_oracle.select(sc, n_kept)
    i64 = idx.astype(np.int64)
    return dict(mu_bar=mu_bar, sigma_bar=sigma_bar, logits=s, scores=sc, kept_idx=idx,
                k_out=np.take_along_axis(np.asarray(k_q8), i64[..., None], axis=2),
                v_out=np.take_along_axis(np.asarray(v_q8), i64[..., None], axis=2),
                v_scale_out=np.take_along_axis(np.asarray(v_scale), i64, axis=2))


def gather_adaptive(k_q8, v_q8, v_scale, idx, offsets):
    """Compaction after head-adaptive eviction (``ea_oracle.select_adaptive``) of a quantised cache: head g of
    unit u owns ``idx[u, offsets[u, g]:offsets[u, g + 1]]``; returns the kept code rows ``[U, B, d]`` (keys,
    values) and the value scales ``[U, B]`` of their tokens, heads one after the other."""
    k_q8, v_q8, v_scale = np.asarray(k_q8), np.asarray(v_q8), np.asarray(v_scale)
    idx, offsets = np.asarray(idx), np.asarray(offsets)
    U, Hkv, n, d = k_q8.shape
    B = idx.shape[1]
    k_out = np.zeros((U, B, d), k_q8.dtype)
    v_out = np.zeros((U, B, d), v_q8.dtype)
    s_out = np.zeros((U, B), v_scale.dtype)
    for u in range(U):
        for g in range(Hkv):
            for j in range(int(offsets[u, g]), int(offsets[u, g + 1])):
                i = int(idx[u, j])
                k_out[u, j], v_out[u, j], s_out[u, j] = k_q8[u, g, i], v_q8[u, g, i], v_scale[u, g, i]
    return k_out, v_out, s_out
