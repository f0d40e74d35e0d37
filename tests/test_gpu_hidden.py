"""GPU parity of the statistics from hidden states (through the C ABI) against the fp64 oracle."""
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


@pytest.mark.parametrize("U,sets,W,dm,Hq,d,layout,cov", [
    (2, 1, 37, 200, 3, 64, 0, 0),        # ragged everywhere: window, d_model (no multiple of 64), 192 columns
    (4, 2, 128, 512, 4, 128, 0, 1),      # two weight sets, units set-major
    (1, 1, 300, 256, 2, 256, 1, 0),      # three window tiles
    (2, 2, 512, 320, 2, 128, 0, 0),      # the largest window
    (3, 3, 1, 64, 1, 64, 0, 0),          # a single buffered state: zero covariance
])
def test_hidden_statistics_match_oracle(ea, oracle, U, sets, W, dm, Hq, d, layout, cov):
    torch.manual_seed(W + dm)
    hidden = (torch.randn(U, W, dm, device="cuda") + 0.5 * torch.randn(U, 1, dm, device="cuda")).to(torch.bfloat16)
    w_q = (torch.randn(sets, Hq * d, dm, device="cuda") / dm ** 0.5).to(torch.bfloat16)
    pos = torch.tensor([1000 + 17 * u for u in range(U)], dtype=torch.int64)
    shape = ea.make_shape(U, Hq, Hq, d, 128, W, rope_layout=layout, cov_norm=cov if W > 1 else 0)
    ctx = ea.Context.for_shape(shape)
    mu_bar, sigma_bar, q = ea.ea_query_stats_hidden(ctx, shape, hidden, w_q, pos.cuda(), 64, 1e4)
    ctx.sync_status()
    # the projected rows themselves: fp32 accumulation of d_model products of bf16 values
    want_q = np.einsum("uwm,ucm->ucw", _widen(hidden), _widen(w_q).repeat(U // sets, axis=0))
    want_q = want_q.reshape(U, Hq, d, W).transpose(0, 1, 3, 2)
    scale = np.sqrt((_widen(hidden) ** 2).sum(-1))[:, None, :, None] * \
        np.sqrt((_widen(w_q).repeat(U // sets, axis=0) ** 2).sum(-1)).reshape(U, Hq, 1, d)
    assert (np.abs(q.cpu().numpy() - want_q) / scale).max() < 2e-6        # |error| <= ~sqrt(dm) 2^-24 |h||w|
    ref_mu, ref_sigma = oracle.query_stats_hidden(inputs.bits(hidden), inputs.bits(w_q), Hq, pos.numpy(), 64, 1e4,
                                                  layout=layout, cov_norm=cov if W > 1 else 0)
    sb = sigma_bar.cpu().numpy().astype(np.float64)
    if W == 1:
        assert np.abs(sb).max() == 0.0
        diag = np.abs(ref_mu) + 1e-30
    else:
        diag = np.sqrt(np.einsum("uhaa->uha", ref_sigma))
        rel = np.abs(sb - ref_sigma) / (diag[..., :, None] * diag[..., None, :] + 1e-30)
        assert rel.max() < 5e-5, rel.max()
        assert np.array_equal(sb, sb.transpose(0, 1, 3, 2))
    mu_err = np.abs(mu_bar.cpu().numpy() - ref_mu) / (diag + np.abs(ref_mu).max(-1, keepdims=True))
    assert mu_err.max() < 5e-5, mu_err.max()


def test_hidden_statistics_feed_the_rest_of_the_path(ea, oracle):
    """Selector projections make q = the hidden channels: same scores as the window-query entry point
    up to the bf16 rounding that entry point's input carries (none here: the channels are bf16)."""
    cfg = inputs.CONFIGS[0].tempered(2.0)
    q_win, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    U, Hq, W, d = q_win.shape
    hidden = q_win.permute(0, 2, 1, 3).reshape(U, W, Hq * d).contiguous()
    w_q = torch.eye(Hq * d, device="cuda", dtype=torch.bfloat16)[None]
    shape = ea.make_shape(U, Hq, cfg.n_kv_heads, d, cfg.n_keys, W)
    ctx = ea.Context.for_shape(shape)
    mu1, sg1 = ea.ea_query_stats(ctx, shape, q_win, pos.cuda(), cfg.n_future, cfg.rope_base)
    mu2, sg2, _ = ea.ea_query_stats_hidden(ctx, shape, hidden, w_q, pos.cuda(), cfg.n_future, cfg.rope_base)
    ctx.sync_status()
    assert torch.equal(mu1, mu2) and torch.equal(sg1, sg2)


def test_hidden_statistics_invalid_arguments(ea):
    shape = ea.make_shape(2, 2, 2, 64, 128, 16)
    ctx = ea.Context.for_shape(shape)
    pos = torch.zeros(2, dtype=torch.int64, device="cuda")
    h = torch.zeros(2, 16, 100, device="cuda", dtype=torch.bfloat16)      # d_model not a multiple of 8
    w = torch.zeros(1, 128, 100, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(ea.EAError) as e:
        ea.ea_query_stats_hidden(ctx, shape, h, w, pos, 8, 1e4)
    assert e.value.status == 1
    h = torch.zeros(2, 16, 96, device="cuda", dtype=torch.bfloat16)
    w3 = torch.zeros(3, 128, 96, device="cuda", dtype=torch.bfloat16)     # 3 sets do not divide 2 units
    with pytest.raises(ea.EAError) as e:
        ea.ea_query_stats_hidden(ctx, shape, h, w3, pos, 8, 1e4)
    assert e.value.status == 1
    big = ea.make_shape(1, 1, 1, 64, 128, 513)                             # window above 512
    ctx2 = ea.Context.for_shape(big)
    with pytest.raises(ea.EAError) as e:
        ea.ea_query_stats_hidden(ctx2, big, torch.zeros(1, 513, 64, device="cuda", dtype=torch.bfloat16),
                                 torch.zeros(1, 64, 64, device="cuda", dtype=torch.bfloat16), pos[:1], 8, 1e4)
    assert e.value.status == 2            # EA_ERR_UNSUPPORTED
