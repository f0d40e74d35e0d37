"""Streaming-decode driver of the fp64 CPU oracle: one cache per KV head and one window of recent
queries per query head carried through consecutive compression events.

TEST INFRASTRUCTURE ONLY (see ``ea_oracle.py``).  It follows the decoding set-up of the paper's
"Implementation details" paragraph: the statistics come from a buffer of the most recent ``W``
states (here: pre-RoPE queries), and every so many generated tokens the cache is compressed down
to a fixed budget with the same routine as in prefill (``ea_oracle.compress``, i.e. Eq. 5-9 and the
eviction rule).  Nothing here is arithmetic of its own: appending is concatenation, the window is
"the last W rows pushed", an event is ``compress`` on what the buffers hold.

Parity status: plumbing around pinned functions; pinned itself (``tests/test_oracle_pins.py``) by a
one-event stream reproducing ``compress`` on the concatenated inputs, by the window equalling the
tail of everything pushed, and by the kept rows of consecutive events composing as index maps.
``QuantStreamOracle`` is the same driver on a quantised cache (``ea_quant``): pinned by a one-event
stream reproducing ``ea_quant.compress`` on the concatenated codes and scales, and by a stream with
unit scales walking through the same kept indices as ``StreamOracle`` on the decoded values.
"""
from __future__ import annotations

import numpy as np

from oracle import ea_oracle, ea_quant


def fill_holes(kept_idx, n_kept: int):
    """Unordered in-place compaction as an index map.  ``kept_idx`` [..., n_kept] ascending kept positions of a
    cache of n rows -> ``where`` [..., n_kept]: the original row that ends up at position j when every kept row
    below ``n_kept`` stays where it is and the kept rows at or beyond ``n_kept`` (ascending) move into the
    evicted positions below ``n_kept`` (ascending).  The kept SET is unchanged, only the order is."""
    idx = np.asarray(kept_idx)
    out = np.empty_like(idx)
    flat_in, flat_out = idx.reshape(-1, idx.shape[-1]), out.reshape(-1, idx.shape[-1])
    for h in range(flat_in.shape[0]):
        kept = [int(i) for i in flat_in[h]]
        stay = set(i for i in kept if i < n_kept)
        movers = [i for i in kept if i >= n_kept]
        holes = [p for p in range(n_kept) if p not in stay]
        where = list(range(n_kept))
        for p, src in zip(holes, movers):
            where[p] = src
        flat_out[h] = where
    return out


class StreamOracle:
    """Caches ``k, v`` uint16 [U, Hkv, n, d] (bf16 bit patterns) and pushed queries uint16 [U, Hq, m, d]."""

    def __init__(self, k_bits, v_bits, window: int, budget: int):
        self.k = np.ascontiguousarray(k_bits)
        self.v = np.ascontiguousarray(v_bits)
        self.window, self.budget = int(window), int(budget)
        self.q = None                       # every query row still inside the window, oldest first

    @property
    def n_keys(self) -> int:
        return self.k.shape[2]

    def append(self, k_new_bits, v_new_bits):
        """New pairs go behind the cached ones (they are the most recent positions)."""
        self.k = np.concatenate([self.k, k_new_bits], axis=2)
        self.v = np.concatenate([self.v, v_new_bits], axis=2)

    def push_queries(self, q_new_bits):
        """The window holds the last ``window`` rows pushed (fewer until that many have arrived)."""
        q = q_new_bits if self.q is None else np.concatenate([self.q, q_new_bits], axis=2)
        self.q = np.ascontiguousarray(q[:, :, -self.window:])

    def compress(self, pos_next, n_future, rope_base, eps, group_mode=ea_oracle.GROUP_MEAN_PROB):
        """One event: scores of every cached pair from the window's statistics, keep ``min(n, budget)`` per
        head.  Returns ``ea_oracle.compress``'s dict; the cache is NOT replaced (see ``keep``)."""
        n_kept = min(self.n_keys, self.budget)
        return ea_oracle.compress(self.q, self.k, self.v, np.asarray(pos_next, dtype=np.int64), n_future,
                                  rope_base, eps, n_kept, group_mode=group_mode)

    def keep(self, kept_idx):
        """Replace every head's cache by its rows ``kept_idx`` [U, Hkv, n_kept], in that order."""
        idx = np.asarray(kept_idx)
        self.k = ea_oracle.gather(self.k, idx)
        self.v = ea_oracle.gather(self.v, idx)


class QuantStreamOracle:
    """The same driver on a quantised cache: codes ``k_q8, v_q8`` uint8 [U, Hkv, n, d], one key scale per
    channel ``k_scale`` [U, Hkv, d] that stays with the cache, one value scale per token ``v_scale`` [U, Hkv, n]
    that travels with its row.  New pairs arrive as codes against the cache's key scales."""

    def __init__(self, k_q8, k_scale, v_q8, v_scale, window: int, budget: int):
        self.k = np.ascontiguousarray(k_q8)
        self.v = np.ascontiguousarray(v_q8)
        self.k_scale = np.ascontiguousarray(k_scale)
        self.v_scale = np.ascontiguousarray(v_scale)
        self.window, self.budget = int(window), int(budget)
        self.q = None

    @property
    def n_keys(self) -> int:
        return self.k.shape[2]

    def append(self, k_new_q8, v_new_q8, v_scale_new):
        self.k = np.concatenate([self.k, k_new_q8], axis=2)
        self.v = np.concatenate([self.v, v_new_q8], axis=2)
        self.v_scale = np.concatenate([self.v_scale, v_scale_new], axis=2)

    def push_queries(self, q_new_bits):
        q = q_new_bits if self.q is None else np.concatenate([self.q, q_new_bits], axis=2)
        self.q = np.ascontiguousarray(q[:, :, -self.window:])

    def compress(self, pos_next, n_future, rope_base, eps, group_mode=ea_oracle.GROUP_MEAN_PROB):
        """One event on what the buffers hold: ``ea_quant.compress``'s dict; the cache is NOT replaced."""
        n_kept = min(self.n_keys, self.budget)
        return ea_quant.compress(self.q, self.k, self.k_scale, self.v, self.v_scale,
                                 np.asarray(pos_next, dtype=np.int64), n_future, rope_base, eps, n_kept,
                                 group_mode=group_mode)

    def keep(self, kept_idx):
        """Replace every head's cache by its rows ``kept_idx`` [U, Hkv, n_kept], in that order; the value
        scales follow their rows, the key scales stay."""
        i64 = np.asarray(kept_idx).astype(np.int64)
        self.k = np.take_along_axis(self.k, i64[..., None], axis=2)
        self.v = np.take_along_axis(self.v, i64[..., None], axis=2)
        self.v_scale = np.take_along_axis(self.v_scale, i64, axis=2)
