"""GPU parity of the contribution score with the output projection (Eq. 9 as written) against the oracle."""
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


def _widen(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("sets,dm,Hq,d", [(1, 96, 4, 64), (2, 300, 2, 128), (1, 128, 1, 256)])
def test_gram_matrices(ea, sets, dm, Hq, d):
    torch.manual_seed(dm)
    w_o = (torch.randn(sets, dm, Hq * d, device="cuda") / dm ** 0.5).to(torch.bfloat16)
    ctx = ea.Context(0, 0)
    gram = ea.ea_wo_gram(ctx, w_o, Hq, d)
    ctx.sync_status()
    w = _widen(w_o).reshape(sets, dm, Hq, d)
    want = np.einsum("samc,same->smce", w, w)
    scale = np.sqrt(np.einsum("smcc->smc", want))
    rel = np.abs(gram.cpu().numpy() - want) / (scale[..., :, None] * scale[..., None, :])
    assert rel.max() < dm * 2.0 ** -24            # d_model exact products added in fp32, in order


def _run(ea, oracle, cfg, n_keys, dm, sets, mode=0, layer=0):
    q, k, v, pos = inputs.generate_layer(cfg, layer=layer, device="cuda", n_keys=n_keys)
    U = cfg.batch * sets
    if sets > 1:                                   # several units: repeat the layer's tensors
        q, k, v, pos = (t.repeat(sets, *[1] * (t.dim() - 1)) for t in (q, k, v, pos))
    g = torch.Generator(device="cuda").manual_seed(99)
    w_o = (torch.randn(sets, dm, cfg.n_q_heads * cfg.head_dim, device="cuda", generator=g) / dm ** 0.5)
    w_o = (w_o * torch.logspace(-0.5, 0.5, cfg.n_q_heads * cfg.head_dim, device="cuda")[None, None, :]).to(torch.bfloat16)
    shape = ea.make_shape(U, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, n_keys, cfg.window, group_mode=mode)
    ctx = ea.Context.for_shape(shape)
    mu_bar, sigma_bar = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    gram = ea.ea_wo_gram(ctx, w_o, cfg.n_q_heads, cfg.head_dim)
    scores, norm2, logits = ea.ea_score_wo(ctx, shape, k, v, mu_bar, sigma_bar, gram, cfg.eps, want_logits=True)
    plain = ea.ea_score(ctx, shape, k, v, mu_bar, sigma_bar, cfg.eps)
    ctx.sync_status()
    vb, wb = inputs.bits(v), inputs.bits(w_o)
    # the squared norms themselves
    G = cfg.n_q_heads // cfg.n_kv_heads
    wo = _widen(w_o).reshape(sets, dm, cfg.n_q_heads, cfg.head_dim)
    vv = _widen(v)
    want_n2 = np.empty((U, cfg.n_q_heads, n_keys))
    for u in range(U):
        for h in range(cfg.n_q_heads):
            y = vv[u, h // G] @ wo[u // (U // sets), :, h, :].T
            want_n2[u, h] = (y * y).sum(-1)
    rel = np.abs(norm2.cpu().numpy() - want_n2) / want_n2
    assert rel.max() < 1e-3, rel.max()               # 16-bit matrix operand, fp32 accumulation
    # the score given the GPU's own log-scores: only the new arithmetic is compared
    own = oracle.scores_wo(_widen(logits), vb, wb, cfg.eps, group_mode=mode)
    np.testing.assert_allclose(scores.cpu().numpy(), own, rtol=2e-3)
    return scores, plain, logits, (q, k, v, pos, w_o)


@pytest.mark.parametrize("cfg_id,n_keys,dm,sets,mode", [(0, 512, 96, 1, 0), (0, 1000, 64, 2, 1), (1, 3000, 256, 1, 0),
                                                        (0, 100, 96, 1, 0)])
def test_score_with_output_projection(ea, oracle, cfg_id, n_keys, dm, sets, mode):
    """Tensor-core path (n >= one tile) and the fp32 fallback (n = 100), one and two weight sets."""
    _run(ea, oracle, inputs.CONFIGS[cfg_id].tempered(2.0, 0.02), n_keys, dm, sets, mode)


def test_score_with_output_projection_head_dim_256(ea, oracle):
    """The paired-CTA tensor-core path (head_dim 256) with the value rows as its operand, ragged cache."""
    import dataclasses
    cfg = dataclasses.replace(inputs.CONFIGS[3].tempered(2.0, 0.02), n_layers=1, n_keys=3000, n_kept=375)
    _run(ea, oracle, cfg, 3000, 192, 1)


def test_whole_path_with_output_projection_against_oracle(ea, oracle):
    cfg = inputs.CONFIGS[0].tempered(2.0, 0.02)
    scores, _, _, (q, k, v, pos, w_o) = _run(ea, oracle, cfg, cfg.n_keys, 96, 1)
    mu_bar, sigma_bar = oracle.query_stats(inputs.bits(q), pos.numpy(), cfg.n_future, cfg.rope_base)
    s = oracle.logits(inputs.bits(k), mu_bar, sigma_bar)
    want = oracle.scores_wo(s, inputs.bits(v), inputs.bits(w_o), cfg.eps)
    np.testing.assert_allclose(scores.cpu().numpy(), want, rtol=1e-2)


def test_selector_output_projection_gives_the_value_norm_scores(ea, oracle):
    cfg = inputs.CONFIGS[0].tempered(2.0, 0.02)
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    d, Hq = cfg.head_dim, cfg.n_q_heads
    sel = torch.zeros(2 * d, d, device="cuda")
    sel[:d] = torch.eye(d, device="cuda")
    w_o = sel.repeat(1, Hq)[None].to(torch.bfloat16)            # every head's slice embeds v unchanged
    shape = ea.make_shape(cfg.batch, Hq, cfg.n_kv_heads, d, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    mu_bar, sigma_bar = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    gram = ea.ea_wo_gram(ctx, w_o, Hq, d)
    scores, _ = ea.ea_score_wo(ctx, shape, k, v, mu_bar, sigma_bar, gram, cfg.eps)
    plain = ea.ea_score(ctx, shape, k, v, mu_bar, sigma_bar, cfg.eps)
    ctx.sync_status()
    torch.testing.assert_close(scores, plain, rtol=1e-5, atol=0)


def test_output_projection_invalid_arguments(ea):
    shape = ea.make_shape(2, 2, 2, 64, 256, 16, group_mode=2)
    ctx = ea.Context.for_shape(shape)
    k = torch.zeros(2, 2, 256, 64, device="cuda", dtype=torch.bfloat16)
    mu = torch.zeros(2, 2, 64, device="cuda")
    sg = torch.zeros(2, 2, 64, 64, device="cuda")
    gram = torch.zeros(1, 2, 64, 64, device="cuda")
    with pytest.raises(ea.EAError) as e:
        ea.ea_score_wo(ctx, shape, k, k, mu, sg, gram, 0.02)
    assert e.value.status == 2            # mean-of-logits grouping has no per-head attention
    shape = ea.make_shape(2, 2, 2, 64, 256, 16)
    with pytest.raises(ea.EAError) as e:
        ea.ea_score_wo(ctx, shape, k, k, mu, sg, torch.zeros(3, 2, 64, 64, device="cuda"), 0.02)
    assert e.value.status == 1            # three weight sets do not divide two units
