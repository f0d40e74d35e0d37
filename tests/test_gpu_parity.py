"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on the same bits."""
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


def _shape(ea, cfg, n_units=None, n_keys=None, **kw):
    return ea.make_shape(cfg.n_units if n_units is None else n_units, cfg.n_q_heads, cfg.n_kv_heads,
                         cfg.head_dim, cfg.n_keys if n_keys is None else n_keys, cfg.window, **kw)


def _run_whole_path(ea, oracle, cfg, group_mode=0, sigma_bits=16, layer=0, direct_rtol=None):
    q, k, v, pos = inputs.generate_layer(cfg, layer=layer, device="cuda")
    shape = _shape(ea, cfg, n_units=cfg.batch, group_mode=group_mode)
    ctx = ea.Context.for_shape(shape)
    out = ea.compress(ctx, shape, q, k, v, pos.cuda(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept,
                      want_logits=True)
    ctx.sync_status()
    qb, kb, vb = inputs.bits(q), inputs.bits(k), inputs.bits(v)
    ref = oracle.compress(qb, kb, vb, pos.numpy(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept,
                          group_mode=group_mode)
    report = {}

    # statistics
    sb, sb_ref = out.sigma_bar.cpu().numpy().astype(np.float64), ref["sigma_bar"]
    diag = np.sqrt(np.einsum("uhaa->uha", sb_ref))
    scale = diag[..., :, None] * diag[..., None, :] + 1e-30
    report["sigma_rel_err"] = float((np.abs(sb - sb_ref) / scale).max())
    mu_err = np.abs(out.mu_bar.cpu().numpy() - ref["mu_bar"]) / (diag + 1e-30)
    report["mu_rel_err"] = float(mu_err.max())
    assert report["sigma_rel_err"] < 2e-5 and report["mu_rel_err"] < 2e-5, report

    # P1 log-scores
    delta = parity.logit_error_bound(kb, ref["mu_bar"], ref["sigma_bar"], sigma_bits)
    bad, worst = parity.check_logits(out.logits.cpu().numpy(), ref["logits"], delta)
    report["logit_bad"], report["logit_worst_rel"] = bad, worst
    assert bad == 0, report

    # P2 scores
    lo, hi = parity.score_range(ref["logits"], delta, vb, cfg.eps, group_mode)
    bad, unstable = parity.check_scores(out.scores.cpu().numpy(), lo, hi)
    report["score_bad"], report["score_unstable"] = bad, unstable
    sc_gpu, sc_ref = out.scores.cpu().numpy().astype(np.float64), ref["scores"]
    report["score_worst_rel"] = float((np.abs(sc_gpu - sc_ref) / np.maximum(sc_ref, 1e-300)).max())
    assert bad == 0, report
    assert unstable <= max(8, lo.size // 1000), report
    if direct_rtol is not None:
        # plain relative error against the oracle, no perturbation band
        np.testing.assert_allclose(sc_gpu, sc_ref, rtol=direct_rtol, atol=0.0)

    # P3 kept set, and exactness of the integer work
    idx = out.kept_idx.cpu().numpy()
    missing, present, free = parity.check_kept(idx, lo, hi, cfg.n_kept)
    report["kept_missing"], report["kept_forbidden"], report["kept_free"] = missing, present, free
    report["kept_diff_vs_oracle"] = int((idx != ref["kept_idx"]).any(-1).sum())
    assert missing == 0 and present == 0, report
    own = oracle.select(out.scores.cpu().numpy().astype(np.float64), cfg.n_kept)
    assert np.array_equal(idx, own), "selection is not the exact top-k of the GPU's own scores"
    assert np.array_equal(inputs.bits(out.k_out), oracle.gather(kb, idx))
    assert np.array_equal(inputs.bits(out.v_out), oracle.gather(vb, idx))
    if free == 0:
        assert np.array_equal(idx, ref["kept_idx"])
        assert np.array_equal(inputs.bits(out.k_out), ref["k_out"])
        assert np.array_equal(inputs.bits(out.v_out), ref["v_out"])
    return report


@pytest.mark.parametrize("cfg_id", [0, 1])
def test_whole_path_literal_configs(ea, oracle, cfg_id):
    print(_run_whole_path(ea, oracle, inputs.CONFIGS[cfg_id]))


@pytest.mark.parametrize("cfg_id,scale,eps", [(0, 2.0, 0.02), (0, 3.0, 0.0), (1, 2.0, 0.02), (1, 3.0, 0.0)])
def test_whole_path_tempered(ea, oracle, cfg_id, scale, eps):
    """Milder outliers spread the softmax over many keys: every slot is then held to 1e-2."""
    rep = _run_whole_path(ea, oracle, inputs.CONFIGS[cfg_id].tempered(scale, eps), direct_rtol=1e-2)
    print(rep)
    assert rep["score_unstable"] == 0


@pytest.mark.parametrize("n,scale,eps", [(3000, 20.0, 0.02), (3000, 2.0, 0.02), (4096, 3.0, 0.0), (300, 2.0, 0.02)])
def test_whole_path_head_dim_256(ea, oracle, n, scale, eps):
    """The 128k-context config's geometry (head_dim 256, two query heads per KV head) on a short,
    ragged cache: several key tiles, a partial last tile, and the paired-CTA tensor-core path."""
    import dataclasses
    cfg = dataclasses.replace(inputs.CONFIGS[3].tempered(scale, eps), n_layers=1, n_keys=n, n_kept=n // 8)
    rep = _run_whole_path(ea, oracle, cfg, direct_rtol=1e-2 if scale <= 3.0 else None)
    print(rep)
    if scale <= 3.0:
        assert rep["score_unstable"] == 0


@pytest.mark.parametrize("cfg_id,layer", [(2, 3), (3, 0), (4, 1)])
def test_whole_path_full_size_layer(ea, oracle, cfg_id, layer):
    """One layer of the benchmark workloads at their full sizes (32k keys at head_dim 128, 128k keys
    at head_dim 256, the decode batch with seven query heads per KV head), same shapes and launch
    configuration per layer as the benchmark, every output element checked against the oracle."""
    import dataclasses
    cfg = dataclasses.replace(inputs.CONFIGS[cfg_id], n_layers=1)
    rep = _run_whole_path(ea, oracle, cfg, layer=layer)
    print(rep)


@pytest.mark.parametrize("cfg_id,layer,scale,eps", [(2, 3, 2.0, 0.02), (2, 5, 3.0, 0.0), (3, 0, 2.0, 0.02),
                                                    (3, 1, 3.0, 0.0), (4, 1, 2.0, 0.02), (4, 2, 3.0, 0.0)])
def test_whole_path_full_size_layer_tempered(ea, oracle, cfg_id, layer, scale, eps):
    """The full-size layers again with milder outliers, so that the softmax is spread over many keys:
    the denominator of Eq. 8 is then a real sum over every work unit of a row (256 partials per row on
    the paired path at 128k keys), the mean over seven query heads matters, and every score is held to
    relative 1e-2 against the oracle directly."""
    import dataclasses
    cfg = dataclasses.replace(inputs.CONFIGS[cfg_id].tempered(scale, eps), n_layers=1)
    rep = _run_whole_path(ea, oracle, cfg, layer=layer, direct_rtol=1e-2)
    print(rep)
    assert rep["score_unstable"] == 0


@pytest.mark.parametrize("mode", [1, 2])
def test_group_modes(ea, oracle, mode):
    print(_run_whole_path(ea, oracle, inputs.CONFIGS[0].tempered(2.0), group_mode=mode))


@pytest.mark.parametrize("d,W,T,layout,cov,pos", [(64, 37, 1, 0, 0, 5), (128, 64, 7, 1, 1, 1000),
                                                  (256, 256, 1024, 0, 0, 131072), (64, 1, 3, 1, 0, 0),
                                                  (128, 130, 512, 0, 1, 8192)])
def test_query_stats(ea, oracle, d, W, T, layout, cov, pos):
    torch.manual_seed(d + W)
    U, Hq = 2, 3
    q = (torch.randn(U, Hq, W, d, device="cuda") * 2 + 0.5).to(torch.bfloat16)
    pos_t = torch.tensor([pos, pos + 17], dtype=torch.int64)
    shape = ea.make_shape(U, Hq, 1, d, 0, W, rope_layout=layout, cov_norm=cov)
    ctx = ea.Context.for_shape(shape)
    if W == 1 and cov == 1:
        pytest.skip("sample covariance needs two queries")
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos_t.cuda(), T, 1e4 if d == 64 else 1e6)
    ctx.sync_status()
    mu_r, sig_r = oracle.query_stats(inputs.bits(q), pos_t.numpy(), T, 1e4 if d == 64 else 1e6,
                                     layout=layout, cov_norm=cov)
    sig = sig.cpu().numpy().astype(np.float64)
    assert np.array_equal(sig, sig.transpose(0, 1, 3, 2)), "sigma_bar must be bitwise symmetric"
    tot = np.sqrt(np.einsum("uhaa->uh", sig_r))[..., None, None] ** 2 / d + 1e-12
    assert (np.abs(sig - sig_r) / tot).max() < 1e-4
    np.testing.assert_allclose(mu.cpu().numpy(), mu_r, atol=2e-5 * (1 + np.abs(mu_r).max()))


@pytest.mark.parametrize("n,n_kept", [(1, 1), (7, 3), (129, 129), (1000, 1), (4097, 2048), (8192, 4096),
                                      (5000, 0), (70001, 35000)])
def test_select_compact_exact(ea, oracle, n, n_kept):
    """Integer work: bit-exact against the oracle, with heavy ties and ragged sizes."""
    torch.manual_seed(n)
    U, Hkv, d = 2, 3, 64
    sc = torch.rand(U, Hkv, n, device="cuda")
    sc[0, 0] = (sc[0, 0] * 4).floor() / 4              # few distinct values: many ties at the cut
    sc[0, 1] = 0.25                                    # all equal
    sc[1, 0, ::3] = -sc[1, 0, ::3]                     # negative scores and zeros of both signs
    sc[1, 0, 1::7] = 0.0
    sc[1, 0, 2::7] = -0.0
    k = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1)
    ctx = ea.Context.for_shape(shape)
    idx, ko, vo = ea.ea_select_compact(ctx, shape, sc, n_kept, k, v)
    ctx.sync_status()
    want = oracle.select(sc.cpu().numpy().astype(np.float64), n_kept)
    assert np.array_equal(idx.cpu().numpy(), want)
    assert np.array_equal(inputs.bits(ko), oracle.gather(inputs.bits(k), want))
    assert np.array_equal(inputs.bits(vo), oracle.gather(inputs.bits(v), want))


@pytest.mark.parametrize("d", [128, 256])
def test_gather_wide_rows(ea, oracle, d):
    torch.manual_seed(d)
    U, Hkv, n, n_kept = 1, 2, 777, 300
    sc = torch.rand(U, Hkv, n, device="cuda")
    k = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1)
    ctx = ea.Context.for_shape(shape)
    idx, ko, vo = ea.ea_select_compact(ctx, shape, sc, n_kept, k, v)
    want = oracle.select(sc.cpu().numpy().astype(np.float64), n_kept)
    assert np.array_equal(idx.cpu().numpy(), want)
    assert np.array_equal(inputs.bits(ko), oracle.gather(inputs.bits(k), want))
    assert np.array_equal(inputs.bits(vo), oracle.gather(inputs.bits(v), want))


@pytest.mark.parametrize("n", [1, 7, 129, 1000])
def test_score_ragged_sizes(ea, oracle, n):
    """Key counts that are not multiples of any tile, down to a single key."""
    cfg = inputs.CONFIGS[0].tempered(2.0)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda", n_keys=n)
    shape = _shape(ea, cfg, n_keys=n)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc, lg = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps, want_logits=True)
    ctx.sync_status()
    mu_r, sig_r = oracle.query_stats(inputs.bits(q), pos.numpy(), cfg.n_future, cfg.rope_base)
    s_r = oracle.logits(inputs.bits(k), mu_r, sig_r)
    sc_r = oracle.scores(s_r, inputs.bits(v), cfg.eps)
    np.testing.assert_allclose(lg.cpu().numpy(), s_r, rtol=1e-4, atol=1e-4)
    np.testing.assert_allclose(sc.cpu().numpy(), sc_r, rtol=1e-2)


@pytest.mark.parametrize("n", [129, 300, 1000])
@pytest.mark.parametrize("d,Hq,Hkv", [(128, 6, 2), (64, 10, 2), (64, 68, 1)])   # the last: more head subsets than the tensor-core kernel takes
def test_score_ragged_sizes_odd_groups(ea, oracle, n, d, Hq, Hkv):
    """Ragged caches with a group size that leaves the last pass of the tensor-core kernel partly
    empty (three query heads per KV head at two heads per pass; five at four per pass)."""
    import dataclasses
    cfg = dataclasses.replace(inputs.CONFIGS[0].tempered(2.0), n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d,
                              window=48, n_keys=n, n_kept=n // 2)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda", n_keys=n)
    shape = _shape(ea, cfg, n_keys=n)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc, lg = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps, want_logits=True)
    ctx.sync_status()
    mu_r, sig_r = oracle.query_stats(inputs.bits(q), pos.numpy(), cfg.n_future, cfg.rope_base)
    s_r = oracle.logits(inputs.bits(k), mu_r, sig_r)
    sc_r = oracle.scores(s_r, inputs.bits(v), cfg.eps)
    delta = parity.logit_error_bound(inputs.bits(k), mu_r, sig_r, 16)
    bad, _ = parity.check_logits(lg.cpu().numpy(), s_r, delta)
    assert bad == 0
    lo, hi = parity.score_range(s_r, delta, inputs.bits(v), cfg.eps, 0)
    bad, unstable = parity.check_scores(sc.cpu().numpy(), lo, hi)
    assert bad == 0 and unstable <= max(8, lo.size // 1000)


def test_decode_events_below_the_budget_keep_every_key(ea, oracle):
    """Streaming decode: while the cache is within its budget (the first events of the schedule) scores
    are still computed but compaction is the identity; the first event above the budget evicts."""
    import dataclasses
    base = inputs.CONFIGS[4]
    events = inputs.decode_schedule()
    for pos, n, kept in (events[0], events[3], events[4]):
        cfg = dataclasses.replace(base, n_layers=1, batch=2, n_keys=n, n_kept=kept)
        q, k, v, _ = inputs.generate_layer(cfg, layer=2, device="cuda", q_phase=0.3)
        pos_next = torch.full((cfg.batch,), pos, dtype=torch.int64)
        shape = _shape(ea, cfg, n_units=cfg.batch)
        ctx = ea.Context.for_shape(shape)
        out = ea.compress(ctx, shape, q, k, v, pos_next.cuda(), cfg.n_future, cfg.rope_base, cfg.eps, kept)
        ctx.sync_status()
        if kept == n:
            want = torch.arange(n, dtype=torch.int32, device="cuda").expand(cfg.batch, cfg.n_kv_heads, n)
            assert torch.equal(out.kept_idx, want)
            assert torch.equal(out.k_out.view(torch.int16), k.view(torch.int16))
            assert torch.equal(out.v_out.view(torch.int16), v.view(torch.int16))
        else:
            ref = oracle.compress(inputs.bits(q), inputs.bits(k), inputs.bits(v), pos_next.numpy(), cfg.n_future,
                                  cfg.rope_base, cfg.eps, kept)
            own = oracle.select(out.scores.cpu().numpy().astype(np.float64), kept)
            assert np.array_equal(out.kept_idx.cpu().numpy(), own)
            agree = (out.kept_idx.cpu().numpy() == ref["kept_idx"]).mean()
            assert agree > 0.99


def test_run_to_run_bitwise_determinism(ea):
    cfg = inputs.CONFIGS[1]
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    shape = _shape(ea, cfg)
    ctx = ea.Context.for_shape(shape)
    a = ea.compress(ctx, shape, q, k, v, pos.cuda(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept)
    b = ea.compress(ctx, shape, q, k, v, pos.cuda(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept)
    ctx.sync_status()
    for x, y in [(a.sigma_bar, b.sigma_bar), (a.scores, b.scores), (a.kept_idx, b.kept_idx)]:
        assert torch.equal(x, y)
    assert torch.equal(a.k_out.view(torch.int16), b.k_out.view(torch.int16))


def test_invalid_arguments_are_rejected_before_launch(ea):
    cfg = inputs.CONFIGS[0]
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    shape = _shape(ea, cfg)
    ctx = ea.Context.for_shape(shape)
    small = ea.Context(0, 256)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)

    def status(fn):
        with pytest.raises(ea.EAError) as e:
            fn()
        return e.value.status

    assert status(lambda: ea.ea_score(small, shape, k, v, mu, sig, cfg.eps)) == 3       # workspace
    assert status(lambda: ea.ea_select_compact(ctx, shape, sc, cfg.n_keys + 1, k, v)) == 1
    assert status(lambda: ea.ea_select_compact(ctx, shape, sc, -1, k, v)) == 1
    assert status(lambda: ea.ea_query_stats(ctx, shape, q, pos.cuda(), 0, cfg.rope_base)) == 1
    bad = ea.make_shape(1, 4, 3, 64, 512, 64)
    assert status(lambda: ea.ea_score(ctx, bad, k, v, mu, sig, cfg.eps)) == 1            # Hq % Hkv
    bad = ea.make_shape(1, 4, 2, 96, 512, 64)
    assert status(lambda: ea.ea_score(ctx, bad, k, v, mu, sig, cfg.eps)) == 2            # head_dim
    # overlapping gather output
    assert status(lambda: ea.ea_select_compact(ctx, shape, sc, 16, k, v, k_out=k, v_out=v)) == 1
    # misaligned key pointer
    with pytest.raises(ea.EAError):
        import ctypes
        ea._check(ea.lib().ea_score(ctx._h, ctypes.byref(shape), ctypes.c_void_p(k.data_ptr() + 2),
                                    ctypes.c_void_p(v.data_ptr()), ctypes.c_void_p(mu.data_ptr()),
                                    ctypes.c_void_p(sig.data_ptr()), 0.02, ctypes.c_void_p(sc.data_ptr()),
                                    None, None), "ea_score")
    # the context still works afterwards
    ctx.sync_status()
    sc2 = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)
    ctx.sync_status()
    assert torch.equal(sc, sc2)


def test_empty_inputs_are_noops(ea):
    shape = ea.make_shape(0, 4, 2, 64, 512, 64)
    ctx = ea.Context(0, 1 << 20)
    assert ea.lib().ea_score(ctx._h, __import__("ctypes").byref(shape), None, None, None, None, 0.02,
                             None, None, None) == 0
    ctx.sync_status()


@pytest.mark.parametrize("chunk", [1, 2, 5])
def test_host_buffer_entry_point_matches_device_calls(ea, chunk):
    """ea_compress_host (host pointers, chunked, copies overlapped) returns the device path's bits."""
    cfg = inputs.CONFIGS[0]
    U = 3
    qs, ks, vs = [], [], []
    for layer in range(U):
        q, k, v, pos = inputs.generate_layer(cfg, layer=layer, device="cuda")
        qs.append(q), ks.append(k), vs.append(v)
    q, k, v = torch.cat(qs), torch.cat(ks), torch.cat(vs)
    pos = torch.tensor([512, 600, 5], dtype=torch.int64)
    shape = _shape(ea, cfg, n_units=U)
    ctx = ea.Context.for_shape(shape)
    want = ea.compress(ctx, shape, q, k, v, pos.cuda(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept)
    ctx.sync_status()
    hctx = ea.Context(0, ea.ea_host_workspace_bytes(shape, cfg.n_kept, chunk))
    hq, hk, hv = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
    hs = torch.empty((U, cfg.n_kv_heads, cfg.n_keys), dtype=torch.float32).pin_memory()
    for _ in range(2):      # twice: staging buffers and events are reused
        idx, ko, vo = ea.ea_compress_host(hctx, shape, hq, hk, hv, pos, cfg.n_future, cfg.rope_base, cfg.eps,
                                          cfg.n_kept, chunk, scores=hs)
        hctx.sync_status()
        assert torch.equal(idx, want.kept_idx.cpu())
        assert torch.equal(ko.view(torch.int16), want.k_out.cpu().view(torch.int16))
        assert torch.equal(vo.view(torch.int16), want.v_out.cpu().view(torch.int16))
        assert torch.equal(hs, want.scores.cpu())
    small = ea.Context(0, 1024)
    with pytest.raises(ea.EAError) as e:
        ea.ea_compress_host(small, shape, hq, hk, hv, pos, cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept, chunk)
    assert e.value.status == 3


@pytest.mark.parametrize("cfg_id,side,budget", [(1, 16, 0), (0, 8, 0), (1, 0, 64), (1, 24, 100)])
def test_side_pass_and_sm_budget_leave_the_result_unchanged(ea, cfg_id, side, budget):
    """The value-norm pass on SMs of its own (ea_set_side_sms) and a log-score kernel limited to part of
    the device (ea_set_sm_budget) are scheduling choices: log-scores bitwise equal, scores equal up to the
    rounding of the norm's square root, same kept set on ties-free data."""
    cfg = inputs.CONFIGS[cfg_id].tempered(2.0)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    shape = _shape(ea, cfg)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    sc0, lg0 = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps, want_logits=True)
    sc0, lg0 = sc0.clone(), lg0.clone()
    ctx.set_side_sms(side)
    ctx.set_sm_budget(budget)
    for _ in range(2):
        sc1, lg1 = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps, want_logits=True)
        ctx.sync_status()
        assert torch.equal(lg0, lg1)
        torch.testing.assert_close(sc1, sc0, rtol=1e-6, atol=0.0)
    ctx.set_side_sms(0)
    ctx.set_sm_budget(0)
    sc2 = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)
    ctx.sync_status()
    assert torch.equal(sc2, sc0)
    for bad in (3, -2, 1000):
        with pytest.raises(ea.EAError):
            ctx.set_side_sms(bad)
    with pytest.raises(ea.EAError):
        ctx.set_sm_budget(16)
