"""Quantised cache (FP8 E4M3 codes with scales) through the C ABI against the quantised oracle."""
import dataclasses

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
    binding.lib()
    return binding


def _np(t):
    return t.detach().cpu().numpy()


@pytest.mark.parametrize("cfg_id,scale,eps,n,mode", [(0, 2.0, 0.02, None, 0), (1, 2.0, 0.02, None, 0), (1, 3.0, 0.0, None, 0),
                                                     (1, 20.0, 0.02, None, 0), (0, 2.0, 0.02, 100, 0), (3, 2.0, 0.02, 3000, 0),
                                                     (0, 2.0, 0.02, None, 1), (0, 2.0, 0.02, None, 2),
                                                     (2, 2.0, 0.02, 32768, 0), (4, 3.0, 0.0, 4608, 0),   # full-size layers, codes widened in the kernel
                                                     (3, 3.0, 0.0, 3000 + 256, 0), (3, 2.0, 0.02, 131072, 0)])
def test_quantised_whole_path(ea, oracle, cfg_id, scale, eps, n, mode):
    """Window statistics, scores of the quantised cache and compaction of code rows with their value scales,
    against the fp64 oracle on the same codes and scales: log-scores and scores within the tolerance protocol
    (and scores to relative 1e-2 directly where the softmax is spread), the kept set against the oracle's
    ranges and bit-exactly against the oracle's selection on the GPU's own scores, gathered codes and scales
    bit-exactly."""
    from oracle import ea_quant
    cfg = inputs.CONFIGS[cfg_id].tempered(scale, eps)
    if n is not None:
        cfg = dataclasses.replace(cfg, n_layers=1, n_keys=n, n_kept=n // 2)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    kq, ks, vq, vs = inputs.quantize_e4m3(k, v)
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window, group_mode=mode)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc, lg = ea.ea_score_q8(ctx, shape, kq, ks, vq, vs, mu, sig, cfg.eps, want_logits=True)
    idx, ko, vo, vso = ea.ea_select_compact_q8(ctx, shape, sc, cfg.n_kept, kq, vq, vs)
    ctx.sync_status()
    ref = ea_quant.compress(inputs.bits(q), _np(kq), _np(ks), _np(vq), _np(vs), pos.numpy(), cfg.n_future, cfg.rope_base,
                            cfg.eps, cfg.n_kept, group_mode=mode)
    k_real, v_real = ea_quant.dequant_k(_np(kq), _np(ks)), ea_quant.dequant_v(_np(vq), _np(vs))
    delta = parity.logit_error_bound(None, ref["mu_bar"], ref["sigma_bar"], 16, k_values=k_real)
    bad, worst = parity.check_logits(_np(lg), ref["logits"], delta)
    assert bad == 0, (bad, worst)
    lo, hi = parity.score_range(ref["logits"], delta, None, cfg.eps, mode, v_values=v_real)
    bad, unstable = parity.check_scores(_np(sc), lo, hi)
    assert bad == 0
    if scale <= 3.0:
        assert unstable == 0
        np.testing.assert_allclose(_np(sc), ref["scores"], rtol=1e-2, atol=0.0)
    else:
        assert unstable <= max(8, lo.size // 1000)
    got = _np(idx)
    missing, present, free = parity.check_kept(got, lo, hi, cfg.n_kept)
    assert missing == 0 and present == 0
    assert np.array_equal(got, oracle.select(_np(sc).astype(np.float64), cfg.n_kept))
    i64 = got.astype(np.int64)
    assert np.array_equal(_np(ko), np.take_along_axis(_np(kq), i64[..., None], axis=2))
    assert np.array_equal(_np(vo), np.take_along_axis(_np(vq), i64[..., None], axis=2))
    assert np.array_equal(_np(vso), np.take_along_axis(_np(vs), i64, axis=2))
    print(dict(logit_worst_rel=worst, free=free,
               score_worst_rel=float((np.abs(_np(sc) - ref["scores"]) / np.maximum(ref["scores"], 1e-300)).max())))


@pytest.mark.parametrize("cfg_id,n", [(0, None), (1, None), (3, 5000), (3, 131072)])
def test_unit_scales_reproduce_the_bf16_path_bitwise(ea, cfg_id, n):
    """With all scales one the quantised entry points see the same numbers as the bf16 ones: same log-scores
    bit for bit (the codes are widened without rounding, the folded scales are ones), at every head_dim the
    tensor-core kernel has a form for."""
    cfg = inputs.CONFIGS[cfg_id].tempered(2.0)
    if n is not None:
        cfg = dataclasses.replace(cfg, n_layers=1, n_keys=n, n_kept=n // 2)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    kq, ks, vq, vs = inputs.quantize_e4m3(k, v)
    ks.fill_(1.0), vs.fill_(1.0)
    k16 = kq.view(torch.float8_e4m3fn).to(torch.bfloat16)
    v16 = vq.view(torch.float8_e4m3fn).to(torch.bfloat16)
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc8, lg8 = ea.ea_score_q8(ctx, shape, kq, ks, vq, vs, mu, sig, cfg.eps, want_logits=True)
    sc8, lg8 = sc8.clone(), lg8.clone()
    sc16, lg16 = ea.ea_score(ctx, shape, k16, v16, mu, sig, cfg.eps, want_logits=True)
    ctx.sync_status()
    assert torch.equal(lg8, lg16)
    torch.testing.assert_close(sc8, sc16, rtol=1e-6, atol=0.0)


def test_quantised_calls_validate_their_arguments(ea):
    cfg = inputs.CONFIGS[0]
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    kq, ks, vq, vs = inputs.quantize_e4m3(k, v)
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc = ea.ea_score_q8(ctx, shape, kq, ks, vq, vs, mu, sig, cfg.eps)
    full = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window,
                         kv_capacity=cfg.n_keys)
    with pytest.raises(ea.EAError) as e:                 # no room behind the cached rows
        ea.ea_cache_append_q8(ctx, full, kq, vq, vs, kq[:, :, :4].contiguous(), vq[:, :, :4].contiguous(),
                              vs[:, :, :4].contiguous())
    assert e.value.status == 1
    with pytest.raises(ea.EAError) as e:                 # K and V must be distinct buffers
        ea.ea_select_compact_inplace_q8(ctx, shape, sc, 8, kq, kq, vs)
    assert e.value.status == 1
    with pytest.raises(ea.EAError) as e:
        ea.ea_select_compact_q8(ctx, shape, sc, cfg.n_keys + 1, kq, vq, vs)
    assert e.value.status == 1
    with pytest.raises(ea.EAError) as e:
        ea.ea_score_q8(ea.Context(0, 256), shape, kq, ks, vq, vs, mu, sig, cfg.eps)
    assert e.value.status == 3
    ctx.sync_status()


@pytest.mark.parametrize("unordered", [False, True])
def test_quantised_cache_carried_through_consecutive_events(ea, oracle, unordered):
    """Streaming decode on ONE buffer of codes: every event appends new code rows (coded against the cache's
    key scales) with their value scales, pushes queries into the window ring, scores the cache inside its
    larger buffer and compacts codes and value scales in place, in temporal order or with the evicted
    positions filled.  Event by event against the oracle's quantised streaming driver on the same codes:
    log-scores and scores within the tolerance protocol (scores to relative 1e-2 directly), the kept set against
    the oracle's ranges and bit-exactly against the oracle's selection on the GPU's own scores, then codes and
    scales of the cache bit-exactly.  The oracle's cache continues from the rows the GPU kept, in the GPU's
    order."""
    from oracle.ea_stream import QuantStreamOracle, fill_holes
    base = inputs.CONFIGS[4].tempered(2.0)
    budget, every, n0 = 1024, 384, 640
    cap = budget + every
    cfg = dataclasses.replace(base, n_layers=1, batch=2, n_keys=n0, n_kept=budget)
    U, Hq, Hkv, d, W = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window
    dev = torch.device("cuda")
    _, k0, v0, _ = inputs.generate_layer(cfg, layer=5, device=dev, n_keys=n0, draw=1)
    kq0, ks, vq0, vs0 = inputs.quantize_e4m3(k0, v0)
    kq = torch.zeros((U, Hkv, cap, d), dtype=torch.uint8, device=dev)
    vq = torch.zeros_like(kq)
    vs = torch.zeros((U, Hkv, cap), dtype=torch.float32, device=dev)
    kq[:, :, :n0], vq[:, :, :n0], vs[:, :, :n0] = kq0, vq0, vs0
    ring = torch.zeros((U, Hq, W, d), dtype=torch.bfloat16, device=dev)
    pushed = torch.zeros((U,), dtype=torch.int64, device=dev)
    st = QuantStreamOracle(_np(kq0), _np(ks), _np(vq0), _np(vs0), window=W, budget=budget)
    ctx = ea.Context.for_shape(ea.make_shape(U, Hq, Hkv, d, cap, W, kv_capacity=cap))
    n_cur, position = n0, n0
    for e, m in enumerate((100, 200, 384, 384)):
        n = n_cur + every
        n_kept = min(n, budget)
        position += every
        _, kn, vn, _ = inputs.generate_layer(cfg, layer=5, device=dev, n_keys=every, draw=2 + e,
                                             key_positions=torch.arange(position - every, position))
        kqn, _, vqn, vsn = inputs.quantize_e4m3(kn, vn, k_scale=ks)
        qn, _, _, _ = inputs.generate_layer(dataclasses.replace(cfg, window=m), layer=5, device=dev, n_keys=1,
                                            draw=100 + e, q_phase=0.1 * e)
        pos = torch.full((U,), position, dtype=torch.int64, device=dev)
        shape_old = ea.make_shape(U, Hq, Hkv, d, n_cur, W, kv_capacity=cap)
        shape = ea.make_shape(U, Hq, Hkv, d, n, W, kv_capacity=cap)
        ea.ea_cache_append_q8(ctx, shape_old, kq, vq, vs, kqn, vqn, vsn)
        ea.ea_window_push(ctx, shape, ring, pushed, qn)
        mu, sigma = ea.ea_query_stats_ring(ctx, shape, ring, pushed, pos, cfg.n_future, cfg.rope_base)
        sc_t, lg_t = ea.ea_score_q8(ctx, shape, kq, ks, vq, vs, mu, sigma, cfg.eps, want_logits=True)
        idx = ea.ea_select_compact_inplace_q8(ctx, shape, sc_t, n_kept, kq, vq, vs, unordered=unordered)
        ctx.sync_status()

        st.append(_np(kqn), _np(vqn), _np(vsn))
        st.push_queries(inputs.bits(qn))
        ref = st.compress(np.full((U,), position), cfg.n_future, cfg.rope_base, cfg.eps)
        from oracle import ea_quant
        k_real, v_real = ea_quant.dequant_k(st.k, st.k_scale), ea_quant.dequant_v(st.v, st.v_scale)
        delta = parity.logit_error_bound(None, ref["mu_bar"], ref["sigma_bar"], 16, k_values=k_real)
        bad, _ = parity.check_logits(_np(lg_t), ref["logits"], delta)
        assert bad == 0, f"event {e}: {bad} log-scores off"
        lo, hi = parity.score_range(ref["logits"], delta, None, cfg.eps, 0, v_values=v_real)
        sc = _np(sc_t)
        bad, unstable = parity.check_scores(sc, lo, hi)
        assert bad == 0 and unstable == 0, f"event {e}"
        np.testing.assert_allclose(sc, ref["scores"], rtol=1e-2, atol=0.0)
        got = _np(idx)
        sel = oracle.select(sc.astype(np.float64), n_kept)                 # ascending kept positions
        missing, present, _ = parity.check_kept(np.sort(got, axis=-1), lo, hi, n_kept)
        assert missing == 0 and present == 0, f"event {e}"
        want = fill_holes(sel, n_kept) if unordered else sel
        assert np.array_equal(got, want), f"event {e}"
        st.keep(got)
        assert np.array_equal(_np(kq[:, :, :n_kept]), st.k), f"event {e}: key codes differ"
        assert np.array_equal(_np(vq[:, :, :n_kept]), st.v), f"event {e}: value codes differ"
        assert np.array_equal(_np(vs[:, :, :n_kept]), st.v_scale), f"event {e}: value scales differ"
        n_cur = n_kept


@pytest.mark.parametrize("cfg_id,floor_share,cap_extra", [(1, 0.2, 0), (0, 0.0, 24), (3, 0.5, 0)])
def test_head_adaptive_eviction_on_a_quantised_cache(ea, oracle, cfg_id, floor_share, cap_extra):
    """Scores of the quantised cache from the CUDA path, then head-adaptive eviction on the code rows: offsets,
    indices, gathered codes and value scales bit-exact against the oracle's routines on the GPU's own scores
    (also with the cache inside a larger buffer)."""
    from oracle import ea_quant
    cfg = inputs.CONFIGS[cfg_id].tempered(2.0, 0.02)
    if cfg_id == 3:
        cfg = dataclasses.replace(cfg, n_layers=1, n_keys=3000, n_kept=700)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    kq, ks, vq, vs = inputs.quantize_e4m3(k, v)
    n, cap = cfg.n_keys, cfg.n_keys + cap_extra
    if cap_extra:
        grow = lambda t: torch.cat([t, torch.zeros_like(t[:, :, :cap_extra])], dim=2).contiguous()
        kq, vq, vs = grow(kq), grow(vq), grow(vs)
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, n, cfg.window, kv_capacity=cap if cap_extra else 0)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc = ea.ea_score_q8(ctx, shape, kq, ks, vq, vs, mu, sig, cfg.eps)
    n_floor = ea.ea_n_floor(cfg.n_kept, floor_share)
    idx, off, ko, vo, so = ea.ea_select_compact_adaptive_q8(ctx, shape, sc, cfg.n_kept, n_floor, kq, vq, vs)
    ctx.sync_status()
    want_idx, want_off = oracle.select_adaptive(_np(sc).astype(np.float64), cfg.n_kept, n_floor)
    assert np.array_equal(_np(off), want_off) and np.array_equal(_np(idx), want_idx)
    wk, wv, ws = ea_quant.gather_adaptive(_np(kq)[:, :, :n], _np(vq)[:, :, :n], _np(vs)[:, :, :n], want_idx, want_off)
    assert np.array_equal(_np(ko), wk) and np.array_equal(_np(vo), wv) and np.array_equal(_np(so), ws)
