"""Tolerance protocol for comparing the CUDA path with the fp64 oracle.

The target is relative error 1e-2 on scores for bf16 inputs with fp32
accumulation.  A softmax turns an ABSOLUTE error of the log-score into a
RELATIVE error of the attention weight, and the synthetic activations reach
log-scores of 1e4..1e5, where no fp32 computation can resolve 1e-2 absolute.
So the comparison is made against the set of results reachable when every
log-score moves by at most ``delta`` (a bound on the CUDA path's log-score
error derived from its arithmetic, see ``logit_error_bound``):

  P1  log-scores:  |s_gpu - s_or| <= min(1e-2 * max(|s_or|, 1), delta)
  P2  scores:      lo * (1 - 1e-2) <= score_gpu <= hi * (1 + 1e-2), where [lo, hi]
                   is the oracle score's range under the log-score perturbation.
                   Where delta is negligible this IS relative error 1e-2.
  P3  kept set:    an index is required when fewer than n_kept others could
                   out-rank it under P2's ranges, forbidden when at least n_kept
                   others certainly out-rank it; the rest may differ.
Selection and compaction themselves are integer work and are checked
bit-exactly against the oracle's selection run on the GPU's own fp32 scores.
"""
from __future__ import annotations

import numpy as np

REL_TOL = 1e-2


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def logit_error_bound(k_bits, mu_bar, sigma_bar, sigma_operand_bits: int, k_values=None):
    """Per (unit, query head, key) bound on the CUDA path's log-score error.

    Three sources, added:
      * fp32 accumulation of the score: 2^-20 of the sum of the magnitudes of its terms;
      * the covariance operand rounded to ``sigma_operand_bits`` significant bits (8 for bf16,
        24 for fp32): each product k_a k_b Sigma_ab carries an independent relative error of at
        most 2^-bits, and six standard deviations of their sum bound the total;
      * the fp32 statistics themselves: each Sigma_ab is off by about 2^-20 sqrt(Sigma_aa
        Sigma_bb) (W fp32 additions), again six standard deviations of the summed effect,
        6 * 2^-20 * sum_a k_a^2 Sigma_aa / (2d).
    """
    k = bf16_to_f64(k_bits) if k_values is None else np.asarray(k_values, dtype=np.float64)   # [U, Hkv, n, d]
    U, Hkv, n, d = k.shape
    Hq = mu_bar.shape[1]
    G = Hq // Hkv
    out = np.empty((U, Hq, n))
    for u in range(U):
        for h in range(Hq):
            kk = k[u, h // G]
            ak, aS = np.abs(kk), np.abs(sigma_bar[u, h])
            absq = ((ak @ aS) * ak).sum(-1) / (2 * d)
            absl = ak @ np.abs(mu_bar[u, h]) / np.sqrt(d)
            k2 = kk ** 2
            rnd = np.sqrt(((k2 @ sigma_bar[u, h] ** 2) * k2).sum(-1)) / (2 * d)
            stat = 6.0 * 2.0 ** -20 * (k2 @ np.diag(sigma_bar[u, h])) / (2 * d)
            out[u, h] = (2.0 ** -20 * (absq + absl) + 6.0 * 2.0 ** (-sigma_operand_bits) / np.sqrt(3) * rnd
                         + stat)
    return out


def check_logits(s_gpu, s_or, delta):
    err = np.abs(s_gpu.astype(np.float64) - s_or)
    tol = np.minimum(REL_TOL * np.maximum(np.abs(s_or), 1.0), np.maximum(delta, 1e-6))
    bad = err > tol
    return int(bad.sum()), float((err / np.maximum(np.abs(s_or), 1.0)).max())


def attention_range(s, delta):
    """Range of softmax_i(s) when every s_j moves independently by at most delta_j.  [.., n]."""
    m = s.max(-1, keepdims=True)
    up = np.exp(s - m + delta)
    dn = np.exp(s - m - delta)
    hi = up / (up + (dn.sum(-1, keepdims=True) - dn))
    lo = dn / (dn + (up.sum(-1, keepdims=True) - up))
    return lo, hi


def score_range(s_or, delta, v_bits, eps, group_mode=0, v_values=None):
    """[lo, hi] of the oracle score (a + eps) * ||v|| under the log-score perturbation."""
    U, Hq, n = s_or.shape
    Hkv = (v_bits if v_values is None else v_values).shape[1]
    G = Hq // Hkv
    vv = bf16_to_f64(v_bits) if v_values is None else np.asarray(v_values, dtype=np.float64)
    vnorm = np.sqrt((vv ** 2).sum(-1))                        # [U, Hkv, n]
    if group_mode == 2:
        s_g = s_or.reshape(U, Hkv, G, n).mean(2)
        d_g = delta.reshape(U, Hkv, G, n).mean(2)
        lo, hi = attention_range(s_g, d_g)
    else:
        lo, hi = attention_range(s_or, delta)
        lo = lo.reshape(U, Hkv, G, n).sum(2)
        hi = hi.reshape(U, Hkv, G, n).sum(2)
        if group_mode == 0:
            lo, hi = lo / G, hi / G
    return (lo + eps) * vnorm, (hi + eps) * vnorm


def check_scores(score_gpu, lo, hi):
    g = score_gpu.astype(np.float64)
    bad = (g < lo * (1 - REL_TOL) - 1e-30) | (g > hi * (1 + REL_TOL) + 1e-30)
    unstable = (hi - lo) > REL_TOL * lo
    return int(bad.sum()), int(unstable.sum())


def check_kept(idx_gpu, lo, hi, n_kept):
    """P3 per head.  Returns (#required indices missing, #forbidden indices present, #free)."""
    lo_t, hi_t = lo * (1 - REL_TOL), hi * (1 + REL_TOL)
    missing = present = free = 0
    heads = lo.reshape(-1, lo.shape[-1]).shape[0]
    lo_f, hi_f = lo_t.reshape(heads, -1), hi_t.reshape(heads, -1)
    idx_f = idx_gpu.reshape(heads, -1)
    n = lo_f.shape[1]
    for h in range(heads):
        hi_sorted = np.sort(hi_f[h])
        lo_sorted = np.sort(lo_f[h])
        # others that could reach at least lo_i (excluding i itself, whose hi >= lo)
        could_beat = n - np.searchsorted(hi_sorted, lo_f[h], side="left") - 1
        surely_beat = n - np.searchsorted(lo_sorted, hi_f[h], side="right")
        required = could_beat < n_kept
        forbidden = surely_beat >= n_kept
        kept = np.zeros(n, bool)
        kept[idx_f[h]] = True
        missing += int((required & ~kept).sum())
        present += int((forbidden & kept).sum())
        free += int((~required & ~forbidden).sum())
    return missing, present, free
