"""Parity in the launch configuration that bench.py times: every layer of a full-size workload
folded into one call, checked against the oracle on sampled (unit, KV head) problems.

A KV head with the query heads of its group is a self-contained problem (statistics, softmax, top-k
are all per head), so the oracle runs the whole path on the sampled heads alone and every output
element of those heads is compared under the tolerance protocol of tests/parity.py.
"""
import numpy as np
import pytest
import torch

import parity
from paper_2510_00636_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ea():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00636_b200 import binding
    binding.lib()          # raises if libea.so is missing: there is no fallback to hide behind
    return binding


@pytest.mark.parametrize("cfg_id,samples", [(3, [(0, 0), (17, 5), (47, 7)]), (2, [(0, 1), (20, 4), (35, 7)])])
def test_all_layers_in_one_call_sampled_heads(ea, oracle, cfg_id, samples):
    import bench
    cfg = inputs.CONFIGS[cfg_id]
    free, _ = torch.cuda.mem_get_info()
    need = cfg.key_slots * 4 * cfg.head_dim * 1.4
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory")
    dev = torch.device("cuda", 0)
    wl = bench.Workload(cfg, dev, ea)
    ctx = wl.make_ctx(wl.n_units)
    wl.step(ctx, wl.n_units)                      # exactly the calls of one timed step
    ctx.sync_status()
    G = cfg.group
    for u, g in samples:
        hq = slice(g * G, (g + 1) * G)
        qb = inputs.bits(wl.q[u:u + 1, hq])
        kb = inputs.bits(wl.k[u:u + 1, g:g + 1])
        vb = inputs.bits(wl.v[u:u + 1, g:g + 1])
        pos = wl.pos[u:u + 1].cpu().numpy()
        ref = oracle.compress(qb, kb, vb, pos, cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept)
        # statistics
        sb = wl.sigma[u:u + 1, hq].cpu().numpy().astype(np.float64)
        diag = np.sqrt(np.einsum("uhaa->uha", ref["sigma_bar"]))
        rel = np.abs(sb - ref["sigma_bar"]) / (diag[..., :, None] * diag[..., None, :] + 1e-30)
        assert rel.max() < 2e-5
        assert (np.abs(wl.mu[u:u + 1, hq].cpu().numpy() - ref["mu_bar"]) / (diag + 1e-30)).max() < 2e-5
        # scores (P2) and kept set (P3) under the log-score error bound of the 16-bit covariance operand
        delta = parity.logit_error_bound(kb, ref["mu_bar"], ref["sigma_bar"], 16)
        lo, hi = parity.score_range(ref["logits"], delta, vb, cfg.eps, 0)
        got = wl.scores[u:u + 1, g:g + 1].cpu().numpy()
        bad, unstable = parity.check_scores(got, lo, hi)
        assert bad == 0 and unstable <= max(8, lo.size // 1000), (u, g, bad, unstable)
        idx = wl.idx[u:u + 1, g:g + 1].cpu().numpy()
        missing, present, free_idx = parity.check_kept(idx, lo, hi, cfg.n_kept)
        assert missing == 0 and present == 0, (u, g, missing, present)
        # integer work: exact on the GPU's own scores
        own = oracle.select(got.astype(np.float64), cfg.n_kept)
        assert np.array_equal(idx, own)
        assert np.array_equal(inputs.bits(wl.k_out[u:u + 1, g:g + 1]), oracle.gather(kb, own))
        assert np.array_equal(inputs.bits(wl.v_out[u:u + 1, g:g + 1]), oracle.gather(vb, own))
        if free_idx == 0:
            assert np.array_equal(idx, ref["kept_idx"])
    del wl
    torch.cuda.empty_cache()


def test_decode_events_in_one_call_sampled_heads(ea, oracle):
    """The streaming config as bench.py runs it (224 units per call, 28 events on one carried cache): every
    event but the last as the benchmark issues them, then the last one call by call with the cache and the
    window ring snapshotted before scoring; sampled heads of it against the oracle, and the compacted cache
    against the oracle's gather of the snapshot."""
    import bench
    cfg = inputs.CONFIGS[4]
    dev = torch.device("cuda", 0)
    wl = bench.DecodeWorkload(cfg, dev, ea)
    ctx = wl.make_ctx(wl.n_units)
    for e, (pos, n, kept) in enumerate(wl.events[:-1]):
        wl._event(ctx, n, kept, e % len(wl.new_q), wl.pos[e])
    e = len(wl.events) - 1
    pos, n, kept = wl.events[e]
    ph = e % len(wl.new_q)
    shape = wl._shape(n)
    ea.ea_cache_append(ctx, wl._shape(n - wl.every), wl.k, wl.v, wl.new_k[ph], wl.new_v[ph])
    ea.ea_window_push(ctx, shape, wl.ring, wl.pushed, wl.new_q[ph])
    ctx.sync_status()
    assert int(wl.pushed[0]) == cfg.window * len(wl.events)
    samples = [(0, 0), (101, 2), (223, 3)]
    snap = {(u, g): (inputs.bits(wl.k[u:u + 1, g:g + 1, :n]), inputs.bits(wl.v[u:u + 1, g:g + 1, :n])) for u, g in samples}
    scores = torch.empty((wl.n_units, cfg.n_kv_heads, n), device=dev)
    idx = torch.empty((wl.n_units, cfg.n_kv_heads, kept), dtype=torch.int32, device=dev)
    ea.ea_query_stats_ring(ctx, shape, wl.ring, wl.pushed, wl.pos[e], cfg.n_future, cfg.rope_base, wl.mu, wl.sigma)
    ea.ea_score(ctx, shape, wl.k, wl.v, wl.mu, wl.sigma, cfg.eps, scores)
    ea.ea_select_compact_inplace(ctx, shape, scores, kept, wl.k, wl.v, idx)
    ctx.sync_status()
    G = cfg.group
    for u, g in samples:
        hq = slice(g * G, (g + 1) * G)
        kb, vb = snap[(u, g)]
        qb = inputs.bits(wl.ring[u:u + 1, hq])
        ref = oracle.compress(qb, kb, vb, np.array([pos], np.int64), cfg.n_future, cfg.rope_base, cfg.eps, kept)
        delta = parity.logit_error_bound(kb, ref["mu_bar"], ref["sigma_bar"], 16)
        lo, hi = parity.score_range(ref["logits"], delta, vb, cfg.eps, 0)
        got = scores[u:u + 1, g:g + 1].cpu().numpy()
        bad, unstable = parity.check_scores(got, lo, hi)
        assert bad == 0 and unstable <= max(8, lo.size // 1000), (u, g, bad, unstable)
        own_idx = idx[u:u + 1, g:g + 1].cpu().numpy()
        missing, present, _ = parity.check_kept(own_idx, lo, hi, kept)
        assert missing == 0 and present == 0, (u, g, missing, present)
        own = oracle.select(got.astype(np.float64), kept)
        assert np.array_equal(own_idx, own)
        assert np.array_equal(inputs.bits(wl.k[u:u + 1, g:g + 1, :kept]), oracle.gather(kb, own))
        assert np.array_equal(inputs.bits(wl.v[u:u + 1, g:g + 1, :kept]), oracle.gather(vb, own))
    del wl
    torch.cuda.empty_cache()
