"""In-place compaction and CUDA-graph capture of a compression event (the decoding set-up)."""
import numpy as np
import pytest
import torch

from paper_2510_00636_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ea():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00636_b200 import binding
    binding.lib()          # raises if libea.so is missing: there is no fallback to hide behind
    return binding


@pytest.mark.parametrize("n,n_kept,d", [(1, 1, 64), (7, 3, 64), (129, 129, 128), (1000, 1, 128), (4608, 4096, 128),
                                        (5000, 0, 64), (3001, 1500, 256), (70001, 35000, 64)])
def test_inplace_compaction_exact(ea, oracle, n, n_kept, d):
    torch.manual_seed(n)
    U, Hkv = 2, 3
    sc = torch.rand(U, Hkv, n, device="cuda")
    sc[0, 0] = (sc[0, 0] * 4).floor() / 4               # many ties at the cut
    sc[0, 1] = torch.arange(n, 0, -1, device="cuda")    # the first n_kept rows stay where they are
    sc[1, 0] = torch.arange(n, device="cuda")           # the last n_kept rows move to the front
    k = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    k0, v0 = inputs.bits(k), inputs.bits(v)
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1)
    ctx = ea.Context.for_shape(shape)
    idx = ea.ea_select_compact_inplace(ctx, shape, sc, n_kept, k, v)
    ctx.sync_status()
    want = oracle.select(sc.cpu().numpy().astype(np.float64), n_kept)
    assert np.array_equal(idx.cpu().numpy(), want)
    k1, v1 = inputs.bits(k), inputs.bits(v)
    assert np.array_equal(k1[:, :, :n_kept], oracle.gather(k0, want))
    assert np.array_equal(v1[:, :, :n_kept], oracle.gather(v0, want))
    assert np.array_equal(k1[:, :, n_kept:], k0[:, :, n_kept:])      # the tail is left alone
    assert np.array_equal(v1[:, :, n_kept:], v0[:, :, n_kept:])


def test_inplace_rejects_overlapping_buffers(ea):
    shape = ea.make_shape(1, 1, 1, 64, 16, 1)
    ctx = ea.Context.for_shape(shape)
    kv = torch.zeros(1, 1, 16, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(ea.EAError) as e:
        ea.ea_select_compact_inplace(ctx, shape, torch.rand(1, 1, 16, device="cuda"), 4, kv, kv)
    assert e.value.status == 1


def test_compression_event_replays_as_a_cuda_graph(ea, oracle):
    """ea_query_stats + ea_score + ea_select_compact_inplace captured once and replayed on new data of
    the same shape: every output is bitwise the one of the eager calls, and matches the oracle's
    selection on the GPU's own scores."""
    cfg = inputs.CONFIGS[0].tempered(2.0)
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    dev = torch.device("cuda")
    data = [inputs.generate_layer(cfg, layer=layer, device=dev) for layer in range(3)]
    q, k, v = (torch.empty_like(t) for t in data[0][:3])
    pos = torch.empty_like(data[0][3], device=dev)
    mu = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), device=dev)
    sigma = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim, cfg.head_dim), device=dev)
    scores = torch.empty((cfg.batch, cfg.n_kv_heads, cfg.n_keys), device=dev)
    idx = torch.empty((cfg.batch, cfg.n_kv_heads, cfg.n_kept), dtype=torch.int32, device=dev)

    def event():
        ea.ea_query_stats(ctx, shape, q, pos, cfg.n_future, cfg.rope_base, mu, sigma)
        ea.ea_score(ctx, shape, k, v, mu, sigma, cfg.eps, scores)
        ea.ea_select_compact_inplace(ctx, shape, scores, cfg.n_kept, k, v, idx)

    def load(layer):
        for dst, src in zip((q, k, v), data[layer][:3]):
            dst.copy_(src)
        pos.copy_(data[layer][3] + 100 * layer)

    eager = []
    for layer in range(3):
        load(layer)
        event()
        ctx.sync_status()
        eager.append([t.clone() for t in (scores, idx, k, v)])

    load(0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        event()                                           # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    load(0)
    # A Context that the garbage collector happens to destroy while the capture is open would call
    # cudaFree, which invalidates a capture: collect what earlier tests left behind first.
    import gc
    gc.collect()
    with torch.cuda.graph(graph):
        event()
    for layer in (1, 2, 0):
        load(layer)
        graph.replay()
        torch.cuda.synchronize()
        for got, want in zip((scores, idx, k, v), eager[layer]):
            assert torch.equal(got, want)
        own = oracle.select(scores.cpu().numpy().astype(np.float64), cfg.n_kept)
        assert np.array_equal(idx.cpu().numpy(), own)
    ctx.sync_status()


def test_one_cache_carried_through_consecutive_events(ea, oracle):
    """Streaming decode on ONE cache buffer and ONE window ring: every event appends the new pairs behind the
    kept ones, pushes the new queries into the ring (partly filled, wrapped, more than a ring at once), takes
    the statistics of what the ring holds, scores the cache at its absolute positions and compacts in place
    to the budget; the last events run as replays of one captured CUDA graph.  Checked event by event against
    the oracle's streaming driver on the same bits: statistics, log-scores and scores within the tolerance
    protocol (every slot stable on these tempered inputs, so scores are held to relative 1e-2 directly), the
    kept set against the oracle's ranges and bit-exactly against the oracle's selection on the GPU's own
    scores, and the cache contents bit-exactly.  So that one borderline index cannot derail the comparison of
    later events, the oracle's cache then continues from the rows the GPU kept (stated in the assertion)."""
    import dataclasses
    import gc
    import parity
    from oracle.ea_stream import StreamOracle
    base = inputs.CONFIGS[4].tempered(2.0)
    budget, every, n0 = 1024, 384, 640
    cap = budget + every
    cfg = dataclasses.replace(base, n_layers=1, batch=2, n_keys=n0, n_kept=budget)
    U, Hq, Hkv, d, W = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window
    dev = torch.device("cuda")
    _, k0, v0, _ = inputs.generate_layer(cfg, layer=3, device=dev, n_keys=n0, draw=1)
    k = torch.zeros((U, Hkv, cap, d), dtype=torch.bfloat16, device=dev)
    v = torch.zeros_like(k)
    k[:, :, :n0], v[:, :, :n0] = k0, v0
    ring = torch.zeros((U, Hq, W, d), dtype=torch.bfloat16, device=dev)
    pushed = torch.zeros((U,), dtype=torch.int64, device=dev)
    st = StreamOracle(inputs.bits(k0), inputs.bits(v0), window=W, budget=budget)
    big = ea.make_shape(U, Hq, Hkv, d, cap, W, kv_capacity=cap)
    ctx = ea.Context.for_shape(big)
    mu = torch.empty((U, Hq, d), device=dev)
    sigma = torch.empty((U, Hq, d, d), device=dev)
    # staging buffers (fixed addresses, so that a captured event can be replayed on new contents)
    k_new, v_new = (torch.empty((U, Hkv, every, d), dtype=torch.bfloat16, device=dev) for _ in range(2))
    q_slots = {m: torch.empty((U, Hq, m, d), dtype=torch.bfloat16, device=dev) for m in (100, 200, 184, 384)}
    pos = torch.empty((U,), dtype=torch.int64, device=dev)
    pushes = [(100,), (200, 184), (384,), (384,), (384,)]          # below a ring, wrapping, more than a ring at once
    n_cur, position = n0, n0
    graph = None
    for e, push in enumerate(pushes):
        n = n_cur + every
        n_kept = min(n, budget)
        position += every
        _, kn, vn, _ = inputs.generate_layer(cfg, layer=3, device=dev, n_keys=every, draw=2 + e,
                                             key_positions=torch.arange(position - every, position))
        k_new.copy_(kn), v_new.copy_(vn)
        q_parts = []
        for i, m in enumerate(push):
            cfg_q = dataclasses.replace(cfg, window=m)
            qn, _, _, _ = inputs.generate_layer(cfg_q, layer=3, device=dev, n_keys=1, draw=100 + 10 * e + i,
                                                q_phase=0.1 * e)
            q_slots[m].copy_(qn)
            q_parts.append(inputs.bits(qn))
        pos.fill_(position)
        shape_old = ea.make_shape(U, Hq, Hkv, d, n_cur, W, kv_capacity=cap)
        shape = ea.make_shape(U, Hq, Hkv, d, n, W, kv_capacity=cap)
        scores = torch.empty((U, Hkv, n), device=dev)
        logits = torch.empty((U, Hq, n), device=dev)
        idx = torch.empty((U, Hkv, n_kept), dtype=torch.int32, device=dev)

        def event():
            ea.ea_cache_append(ctx, shape_old, k, v, k_new, v_new)
            for m in push:
                ea.ea_window_push(ctx, shape, ring, pushed, q_slots[m])
            ea.ea_query_stats_ring(ctx, shape, ring, pushed, pos, cfg.n_future, cfg.rope_base, mu, sigma)
            ea.ea_score(ctx, shape, k, v, mu, sigma, cfg.eps, scores, logits)
            ea.ea_select_compact_inplace(ctx, shape, scores, n_kept, k, v, idx)

        if e < 3:
            event()
        else:
            if graph is None:
                # events 2, 3 and 4 have one shape: capture it once (event 2 already ran it eagerly), replay twice
                gc.collect()
                graph = torch.cuda.CUDAGraph()
                g_scores, g_logits, g_idx = scores, logits, idx
                with torch.cuda.graph(graph):
                    event()
            graph.replay()
            scores, logits, idx = g_scores, g_logits, g_idx
        ctx.sync_status()

        # the oracle's side of the same event
        st.append(inputs.bits(kn), inputs.bits(vn))
        for qb in q_parts:
            st.push_queries(qb)
        ref = st.compress(np.full((U,), position), cfg.n_future, cfg.rope_base, cfg.eps)
        assert int(pushed[0]) == sum(sum(p) for p in pushes[:e + 1])
        sb, sb_ref = sigma.cpu().numpy().astype(np.float64), ref["sigma_bar"]
        dg = np.sqrt(np.einsum("uhaa->uha", sb_ref))
        assert (np.abs(sb - sb_ref) / (dg[..., :, None] * dg[..., None, :] + 1e-30)).max() < 2e-5, f"event {e}"
        assert (np.abs(mu.cpu().numpy() - ref["mu_bar"]) / (dg + 1e-30)).max() < 2e-5, f"event {e}"
        delta = parity.logit_error_bound(st.k, ref["mu_bar"], ref["sigma_bar"], 16)
        bad, _ = parity.check_logits(logits.cpu().numpy(), ref["logits"], delta)
        assert bad == 0, f"event {e}: {bad} log-scores off"
        lo, hi = parity.score_range(ref["logits"], delta, st.v, cfg.eps, 0)
        sc = scores.cpu().numpy()
        bad, unstable = parity.check_scores(sc, lo, hi)
        assert bad == 0 and unstable == 0, f"event {e}"
        np.testing.assert_allclose(sc, ref["scores"], rtol=1e-2, atol=0.0)
        got = idx.cpu().numpy()
        missing, present, free = parity.check_kept(got, lo, hi, n_kept)
        assert missing == 0 and present == 0, f"event {e}"
        assert np.array_equal(got, oracle.select(sc.astype(np.float64), n_kept)), f"event {e}"
        if n_kept == n:
            assert np.array_equal(got, np.broadcast_to(np.arange(n, dtype=np.int32), got.shape))
        # cache contents after the event: the rows the GPU kept, in order, at the front of every head's range;
        # the oracle's cache continues from those rows
        st.keep(got)
        assert np.array_equal(inputs.bits(k[:, :, :n_kept]), st.k), f"event {e}: key cache differs"
        assert np.array_equal(inputs.bits(v[:, :, :n_kept]), st.v), f"event {e}: value cache differs"
        print(f"event {e}: n {n} -> {n_kept}, free indices {free}, differ from oracle's own selection "
              f"{int((got != ref['kept_idx']).any(-1).sum())} heads")
        n_cur = n_kept


def test_ring_statistics_partly_filled_and_wrapped(ea, oracle):
    """ea_query_stats_ring against the oracle's statistics of the last min(pushed, W) rows, for a ring that
    is empty (zero statistics), holds one row, is partly filled, exactly full and wrapped."""
    torch.manual_seed(5)
    U, Hq, d, W = 2, 3, 64, 16
    shape = ea.make_shape(U, Hq, 1, d, 0, W)
    ctx = ea.Context.for_shape(shape)
    ring = torch.zeros((U, Hq, W, d), dtype=torch.bfloat16, device="cuda")
    pushed = torch.zeros((U,), dtype=torch.int64, device="cuda")
    pos = torch.tensor([100, 7], dtype=torch.int64, device="cuda")
    mu, sig = ea.ea_query_stats_ring(ctx, shape, ring, pushed, pos, 8, 1e4)
    ctx.sync_status()
    assert float(mu.abs().max()) == 0.0 and float(sig.abs().max()) == 0.0
    everything = None
    for m in (1, 6, 9, 5, 40):
        q = (torch.randn(U, Hq, m, d, device="cuda") * 2 + 0.5).to(torch.bfloat16)
        ea.ea_window_push(ctx, shape, ring, pushed, q)
        everything = q if everything is None else torch.cat([everything, q], dim=2)
        mu, sig = ea.ea_query_stats_ring(ctx, shape, ring, pushed, pos, 8, 1e4)
        ctx.sync_status()
        tail = inputs.bits(everything[:, :, -W:])
        mu_r, sig_r = oracle.query_stats(tail, pos.cpu().numpy(), 8, 1e4)
        sig = sig.cpu().numpy().astype(np.float64)
        tot = np.sqrt(np.einsum("uhaa->uh", sig_r))[..., None, None] ** 2 / d + 1e-12
        assert (np.abs(sig - sig_r) / tot).max() < 1e-4, m
        np.testing.assert_allclose(mu.cpu().numpy(), mu_r, atol=2e-5 * (1 + np.abs(mu_r).max()))
        assert pushed.tolist() == [everything.shape[2]] * U


@pytest.mark.parametrize("n,n_kept,d,cap", [(1, 1, 64, 0), (7, 3, 64, 9), (129, 129, 128, 0), (1000, 1, 128, 1000), (4608, 4096, 128, 4608),
                                            (3001, 1500, 256, 3100), (30000, 25600, 64, 0)])
def test_unordered_inplace_compaction_exact(ea, oracle, n, n_kept, d, cap):
    """The unordered compaction against the oracle's index map: same kept set as the ordered selection, kept rows
    below n_kept untouched, the others filled from the tail; rows at and beyond n_kept and everything outside
    the heads' ranges are left alone."""
    from oracle.ea_stream import fill_holes
    torch.manual_seed(n)
    U, Hkv = 2, 3
    rows = cap or n
    sc = torch.rand(U, Hkv, n, device="cuda")
    sc[0, 0] = (sc[0, 0] * 4).floor() / 4               # many ties at the cut
    sc[0, 1] = torch.arange(n, 0, -1, device="cuda")    # nothing moves
    sc[1, 0] = torch.arange(n, device="cuda")           # everything kept sits in the tail
    k = torch.randn(U, Hkv, rows, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, rows, d, device="cuda").to(torch.bfloat16)
    k0, v0 = inputs.bits(k), inputs.bits(v)
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1, kv_capacity=cap)
    ctx = ea.Context.for_shape(shape)
    where = ea.ea_select_compact_inplace_unordered(ctx, shape, sc, n_kept, k, v)
    ctx.sync_status()
    want = fill_holes(oracle.select(sc.cpu().numpy().astype(np.float64), n_kept), n_kept)
    assert np.array_equal(where.cpu().numpy(), want)
    k1, v1 = inputs.bits(k), inputs.bits(v)
    assert np.array_equal(k1[:, :, :n_kept], oracle.gather(k0[:, :, :n], want))
    assert np.array_equal(v1[:, :, :n_kept], oracle.gather(v0[:, :, :n], want))
    assert np.array_equal(k1[:, :, n_kept:], k0[:, :, n_kept:]) and np.array_equal(v1[:, :, n_kept:], v0[:, :, n_kept:])


@pytest.mark.parametrize("d,Hq,Hkv,n,ring", [(128, 28, 4, 1408, True), (128, 8, 2, 640, False), (64, 10, 2, 300, False),
                                             (64, 4, 2, 512, True)])
def test_fused_statistics_give_the_same_scores_bit_for_bit(ea, d, Hq, Hkv, n, ring):
    """ea_set_fused_stats: the operand written by the statistics kernel must be, bit for bit, the one
    ea_score builds from mu_bar and sigma_bar - so the log-scores and the scores of
    ea_score(NULL, NULL) equal those of the two-step path exactly, with and without sigma_bar
    written, for a plain window and for a ring (partly filled and wrapped, and empty)."""
    import dataclasses
    cfg = dataclasses.replace(inputs.CONFIGS[4].tempered(2.0), n_layers=1, batch=3, n_q_heads=Hq, n_kv_heads=Hkv,
                              head_dim=d, n_keys=n, window=48)
    q, k, v, pos = inputs.generate_layer(cfg, layer=1, device="cuda")
    U, W = cfg.batch, cfg.window
    shape = ea.make_shape(U, Hq, Hkv, d, n, W)
    ctx = ea.Context.for_shape(shape)
    pos = pos.cuda()
    ringbuf = torch.zeros_like(q)
    pushed = torch.zeros((U,), dtype=torch.int64, device="cuda")

    def stats(**kw):
        if ring:
            return ea.ea_query_stats_ring(ctx, shape, ringbuf, pushed, pos, cfg.n_future, cfg.rope_base, **kw)
        return ea.ea_query_stats(ctx, shape, q, pos, cfg.n_future, cfg.rope_base, **kw)

    for fill in ([0, 20, 70] if ring else [None]):
        if fill:
            ea.ea_window_push(ctx, shape, ringbuf, pushed, q[:, :, :fill - int(pushed[0]) if fill <= W else W].contiguous())
        ctx.set_fused_stats(False)
        mu, sig = stats()
        sc0, lg0 = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps, want_logits=True)
        sc0, lg0 = sc0.clone(), lg0.clone()
        ctx.set_fused_stats(True)
        mu1, sig1 = stats()
        assert torch.equal(mu1, mu) and torch.equal(sig1, sig)
        sc1, lg1 = ea.ea_score(ctx, shape, k, v, None, None, cfg.eps, want_logits=True)
        assert torch.equal(lg1, lg0) and torch.equal(sc1, sc0)
        mu2, none = stats(want_sigma=False)
        assert none is None and torch.equal(mu2, mu)
        sc2, lg2 = ea.ea_score(ctx, shape, k, v, None, None, cfg.eps, want_logits=True)
        ctx.sync_status()
        assert torch.equal(lg2, lg0) and torch.equal(sc2, sc0)
    # a scoring call with explicit statistics rebuilds the images: the fused ones no longer stand
    stats()
    ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)
    with pytest.raises(ea.EAError) as e:
        ea.ea_score(ctx, shape, k, v, None, None, cfg.eps)
    assert e.value.status == 1
    # without a matching operand the call is refused
    other = ea.make_shape(U, Hq, Hkv, d, n - 1 if n > 129 else n + 1, W)
    big = ea.Context.for_shape(ea.make_shape(U, Hq, Hkv, d, n + 1, W))
    with pytest.raises(ea.EAError) as e:
        ea.ea_score(big, other, k[:, :, :other.n_keys].contiguous(), v[:, :, :other.n_keys].contiguous(), None, None, cfg.eps)
    assert e.value.status == 1
    ctx.set_fused_stats(False)
    with pytest.raises(ea.EAError):
        stats(want_sigma=False)
    with pytest.raises(ea.EAError):
        ea.ea_score(ctx, shape, k, v, None, None, cfg.eps)


def test_streaming_calls_validate_their_arguments(ea):
    U, Hq, Hkv, d, W, cap = 1, 4, 2, 64, 8, 40
    k = torch.zeros((U, Hkv, cap, d), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros_like(k)
    new = torch.ones((U, Hkv, 16, d), dtype=torch.bfloat16, device="cuda")
    ring = torch.zeros((U, Hq, W, d), dtype=torch.bfloat16, device="cuda")
    pushed = torch.zeros((U,), dtype=torch.int64, device="cuda")
    ctx = ea.Context.for_shape(ea.make_shape(U, Hq, Hkv, d, cap, W, kv_capacity=cap))

    def status(fn):
        with pytest.raises(ea.EAError) as e:
            fn()
        return e.value.status

    # appending beyond the capacity, and a capacity below the cache length
    assert status(lambda: ea.ea_cache_append(ctx, ea.make_shape(U, Hq, Hkv, d, 30, W, kv_capacity=cap), k, v, new, new)) == 1
    assert status(lambda: ea.ea_cache_append(ctx, ea.make_shape(U, Hq, Hkv, d, 30, W, kv_capacity=20), k, v, new, new)) == 1
    # exactly to the brim is fine, and lands where it should
    ea.ea_cache_append(ctx, ea.make_shape(U, Hq, Hkv, d, 24, W, kv_capacity=cap), k, v, new, new)
    ctx.sync_status()
    assert float(k[:, :, :24].abs().max()) == 0.0 and float(k[:, :, 24:].min()) == 1.0
    # a ring without rows, a missing counter
    assert status(lambda: ea.ea_window_push(ctx, ea.make_shape(U, Hq, Hkv, d, 0, 0), ring, pushed, new[:, :, :4].repeat(1, 2, 1, 1))) == 1
    shape = ea.make_shape(U, Hq, Hkv, d, 0, W)
    import ctypes
    L = ea.lib()
    assert L.ea_window_push(ctx._h, ctypes.byref(shape), ctypes.c_void_p(ring.data_ptr()), None,
                            ctypes.c_void_p(ring.data_ptr()), 2, None) == 1
    assert L.ea_query_stats_ring(ctx._h, ctypes.byref(shape), ctypes.c_void_p(ring.data_ptr()), None, None, 4, 1e4, None,
                                 None, None) == 1
    # empty pushes and appends are no-ops
    ea.ea_window_push(ctx, shape, ring, pushed, ring[:, :, :0].contiguous())
    ctx.sync_status()
    assert int(pushed[0]) == 0


@pytest.mark.parametrize("unordered", [False, True])
def test_value_norms_carried_with_the_cache(ea, oracle, unordered):
    """Streaming decode with the value norms carried beside the cache: norms of the appended rows only
    (ea_value_norms), scores from the norms (ea_score_vnorm), the norms moved like the rows
    (ea_carry_f32_inplace).  Every event: scores within the tolerance protocol of the oracle's streaming driver
    (and to relative 1e-2 directly), equal to ea_score's on the same cache up to the rounding of the sum of
    squares, the kept set exact on the GPU's own scores, and afterwards every carried norm equal to the norm of
    the row it sits beside."""
    import dataclasses
    import parity
    from oracle.ea_stream import StreamOracle, fill_holes
    base = inputs.CONFIGS[4].tempered(2.0)
    budget, every, n0 = 1024, 384, 640
    cap = budget + every
    cfg = dataclasses.replace(base, n_layers=1, batch=2, n_keys=n0, n_kept=budget)
    U, Hq, Hkv, d, W = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window
    dev = torch.device("cuda")
    _, k0, v0, _ = inputs.generate_layer(cfg, layer=7, device=dev, n_keys=n0, draw=1)
    k = torch.zeros((U, Hkv, cap, d), dtype=torch.bfloat16, device=dev)
    v = torch.zeros_like(k)
    k[:, :, :n0], v[:, :, :n0] = k0, v0
    v_norm = torch.full((U, Hkv, cap), float("nan"), device=dev)          # nothing may read a norm never written
    ring = torch.zeros((U, Hq, W, d), dtype=torch.bfloat16, device=dev)
    pushed = torch.zeros((U,), dtype=torch.int64, device=dev)
    st = StreamOracle(inputs.bits(k0), inputs.bits(v0), window=W, budget=budget)
    ctx = ea.Context.for_shape(ea.make_shape(U, Hq, Hkv, d, cap, W, kv_capacity=cap))
    ea.ea_value_norms(ctx, ea.make_shape(U, Hq, Hkv, d, n0, W, kv_capacity=cap), v, 0, n0, v_norm)
    n_cur, position = n0, n0
    for e, m in enumerate((100, 200, 384, 384)):
        n = n_cur + every
        n_kept = min(n, budget)
        position += every
        _, kn, vn, _ = inputs.generate_layer(cfg, layer=7, device=dev, n_keys=every, draw=2 + e,
                                             key_positions=torch.arange(position - every, position))
        qn, _, _, _ = inputs.generate_layer(dataclasses.replace(cfg, window=m), layer=7, device=dev, n_keys=1,
                                            draw=100 + e, q_phase=0.1 * e)
        pos = torch.full((U,), position, dtype=torch.int64, device=dev)
        shape_old = ea.make_shape(U, Hq, Hkv, d, n_cur, W, kv_capacity=cap)
        shape = ea.make_shape(U, Hq, Hkv, d, n, W, kv_capacity=cap)
        ea.ea_cache_append(ctx, shape_old, k, v, kn, vn)
        ea.ea_value_norms(ctx, shape, v, n_cur, every, v_norm)
        ea.ea_window_push(ctx, shape, ring, pushed, qn)
        mu, sigma = ea.ea_query_stats_ring(ctx, shape, ring, pushed, pos, cfg.n_future, cfg.rope_base)
        sc_t, lg_t = ea.ea_score_vnorm(ctx, shape, k, v_norm, mu, sigma, cfg.eps, want_logits=True)
        sc_v = ea.ea_score(ctx, shape, k, v, mu, sigma, cfg.eps)
        torch.testing.assert_close(sc_t, sc_v, rtol=1e-5, atol=0.0)
        compact = ea.ea_select_compact_inplace_unordered if unordered else ea.ea_select_compact_inplace
        idx = compact(ctx, shape, sc_t, n_kept, k, v)
        ea.ea_carry_f32_inplace(ctx, shape, idx, n_kept, v_norm)
        ctx.sync_status()

        st.append(inputs.bits(kn), inputs.bits(vn))
        st.push_queries(inputs.bits(qn))
        ref = st.compress(np.full((U,), position), cfg.n_future, cfg.rope_base, cfg.eps)
        delta = parity.logit_error_bound(st.k, ref["mu_bar"], ref["sigma_bar"], 16)
        bad, _ = parity.check_logits(lg_t.cpu().numpy(), ref["logits"], delta)
        assert bad == 0, f"event {e}"
        lo, hi = parity.score_range(ref["logits"], delta, st.v, cfg.eps, 0)
        sc = sc_t.cpu().numpy()
        bad, unstable = parity.check_scores(sc, lo, hi)
        assert bad == 0 and unstable == 0, f"event {e}"
        np.testing.assert_allclose(sc, ref["scores"], rtol=1e-2, atol=0.0)
        got = idx.cpu().numpy()
        sel = oracle.select(sc.astype(np.float64), n_kept)
        assert np.array_equal(got, fill_holes(sel, n_kept) if unordered else sel), f"event {e}"
        st.keep(got)
        assert np.array_equal(inputs.bits(v[:, :, :n_kept]), st.v), f"event {e}: value cache differs"
        want_norm = v[:, :, :n_kept].float().square().sum(-1).sqrt()
        torch.testing.assert_close(v_norm[:, :, :n_kept], want_norm, rtol=2e-6, atol=0.0)
        n_cur = n_kept
