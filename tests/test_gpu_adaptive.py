"""GPU parity of head-adaptive eviction (through the C ABI) against the fp64 oracle.

Selection and compaction are integer work on given scores: every comparison here is bit-exact.
"""
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


def _check_against_oracle(ea, oracle, sc, n_kept, n_floor, k=None, v=None):
    U, Hkv, n = sc.shape
    d = 64 if k is None else k.shape[-1]
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1)
    ctx = ea.Context.for_shape(shape)
    idx, off, ko, vo = ea.ea_select_compact_adaptive(ctx, shape, sc, n_kept, n_floor, k, v, gather=k is not None)
    ctx.sync_status()
    want_idx, want_off = oracle.select_adaptive(sc.cpu().numpy().astype(np.float64), n_kept, n_floor)
    assert np.array_equal(off.cpu().numpy(), want_off)
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    if k is not None:
        assert np.array_equal(inputs.bits(ko), oracle.gather_adaptive(inputs.bits(k), want_idx, want_off))
        assert np.array_equal(inputs.bits(vo), oracle.gather_adaptive(inputs.bits(v), want_idx, want_off))
    return want_off


@pytest.mark.parametrize("U,Hkv,n,n_kept", [(2, 3, 1000, 400), (1, 1, 257, 100), (3, 2, 7, 3), (1, 8, 40000, 9000),
                                           (2, 4, 16385, 1), (1, 5, 70001, 35000), (1, 2, 1, 1)])
@pytest.mark.parametrize("floor_share", [0.0, 0.2, 1.0])
def test_adaptive_select_exact(ea, oracle, U, Hkv, n, n_kept, floor_share):
    """Heads of different scale, heavy ties at the thresholds, negative scores, zeros of both signs."""
    torch.manual_seed(n + Hkv)
    d = 64
    sc = torch.rand(U, Hkv, n, device="cuda")
    scale = torch.logspace(-1.5, 1.0, Hkv, device="cuda")
    sc = sc * scale[None, :, None]
    sc[0, 0] = (sc[0, 0] * 64).floor() / 64             # few distinct values: ties at both thresholds
    if Hkv > 1:
        sc[0, 1] = sc[0, 0]                              # two heads with the same scores: ties across heads
    if U > 1:
        sc[1, 0, ::3] = -sc[1, 0, ::3]
        sc[1, 0, 1::7] = 0.0
        sc[1, 0, 2::7] = -0.0
    k = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    n_floor = ea.ea_n_floor(n_kept, floor_share)
    assert n_floor == oracle.n_floor(n_kept, floor_share)
    off = _check_against_oracle(ea, oracle, sc, n_kept, n_floor, k, v)
    if floor_share == 1.0:
        assert np.array_equal(off, np.tile(np.arange(Hkv + 1) * n_kept, (U, 1)))


def test_adaptive_all_scores_equal(ea, oracle):
    sc = torch.full((2, 4, 3000), 0.25, device="cuda")
    _check_against_oracle(ea, oracle, sc, 1000, 200)
    _check_against_oracle(ea, oracle, sc, 1000, 0)


@pytest.mark.parametrize("n_kept,n_floor", [(0, 0), (500, 500), (500, 0), (499, 99), (1, 0)])
def test_adaptive_edge_budgets(ea, oracle, n_kept, n_floor):
    torch.manual_seed(5)
    sc = torch.rand(2, 3, 500, device="cuda") * torch.tensor([1.0, 5.0, 0.2], device="cuda")[None, :, None]
    k = torch.randn(2, 3, 500, 128, device="cuda").to(torch.bfloat16)
    v = torch.randn(2, 3, 500, 128, device="cuda").to(torch.bfloat16)
    _check_against_oracle(ea, oracle, sc, n_kept, n_floor, k, v)


def test_adaptive_equals_per_head_selection_when_safeguard_is_the_budget(ea):
    torch.manual_seed(6)
    U, Hkv, n, d, n_kept = 2, 4, 5000, 256, 1234
    sc = torch.rand(U, Hkv, n, device="cuda")
    k = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1)
    ctx = ea.Context.for_shape(shape)
    idx, ko, vo = ea.ea_select_compact(ctx, shape, sc, n_kept, k, v)
    idx2, off, ko2, vo2 = ea.ea_select_compact_adaptive(ctx, shape, sc, n_kept, n_kept, k, v)
    ctx.sync_status()
    assert torch.equal(idx.reshape(U, -1), idx2)
    assert torch.equal(ko.reshape(U, -1, d), ko2) and torch.equal(vo.reshape(U, -1, d), vo2)


def test_adaptive_whole_path_tempered(ea, oracle):
    """Scores from the CUDA path on a config whose softmax is spread out, then head-adaptive eviction:
    bit-exact on the GPU's own scores, and inside the tolerance band of the oracle's whole path."""
    cfg = inputs.CONFIGS[1].tempered(2.0, 0.02)
    q, k, v, pos = inputs.generate_layer(cfg, layer=0, device="cuda")
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    mu_bar, sigma_bar = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    scores = ea.ea_score(ctx, shape, k, v, mu_bar, sigma_bar, cfg.eps)
    n_floor = ea.ea_n_floor(cfg.n_kept, 0.2)
    idx, off, ko, vo = ea.ea_select_compact_adaptive(ctx, shape, scores, cfg.n_kept, n_floor, k, v)
    ctx.sync_status()
    own = scores.cpu().numpy().astype(np.float64)
    want_idx, want_off = oracle.select_adaptive(own, cfg.n_kept, n_floor)
    assert np.array_equal(off.cpu().numpy(), want_off) and np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.array_equal(inputs.bits(ko), oracle.gather_adaptive(inputs.bits(k), want_idx, want_off))
    assert np.array_equal(inputs.bits(vo), oracle.gather_adaptive(inputs.bits(v), want_idx, want_off))
    # against the oracle's own scores: relative score error <= 1e-2 moves every threshold by at most that
    # much, so a pair well above (below) the oracle's thresholds must be kept (dropped)
    ref = oracle.compress(inputs.bits(q), inputs.bits(k), inputs.bits(v), pos.numpy(), cfg.n_future,
                          cfg.rope_base, cfg.eps, cfg.n_kept)
    ref_idx, ref_off = oracle.select_adaptive(ref["scores"], cfg.n_kept, n_floor)
    tol = 2.1e-2
    Hkv, n = cfg.n_kv_heads, cfg.n_keys
    for u in range(cfg.batch):
        sc = ref["scores"][u]
        kept_ref = np.zeros((Hkv, n), bool)
        kept_gpu = np.zeros((Hkv, n), bool)
        for g in range(Hkv):
            kept_ref[g, ref_idx[u, ref_off[u, g]:ref_off[u, g + 1]]] = True
            kept_gpu[g, want_idx[u, want_off[u, g]:want_off[u, g + 1]]] = True
        # thresholds of the oracle: the unit's (lowest score kept beyond a safeguard share) and each head's safeguard
        floor_thr = np.sort(sc, axis=1)[:, ::-1][:, n_floor - 1] if n_floor > 0 else np.full(Hkv, np.inf)
        sizes = np.diff(ref_off[u])
        beyond = [np.sort(sc[g])[::-1][sizes[g] - 1] for g in range(Hkv) if sizes[g] > n_floor]
        unit_thr = min(beyond) if beyond else np.inf
        thr = np.minimum(floor_thr, unit_thr)[:, None]
        assert not (~kept_gpu & (sc > thr * (1 + tol))).any()
        assert not (kept_gpu & (sc < thr * (1 - tol))).any()
        assert (kept_gpu != kept_ref).sum() <= 0.05 * kept_ref.sum()


def test_adaptive_full_size_layer(ea, oracle):
    """One layer of the 128k-token workload's shape (8 heads of 131072 keys, 16384 kept on average)."""
    torch.manual_seed(7)
    Hkv, n, n_kept = 8, 131072, 16384
    g = torch.Generator(device="cuda").manual_seed(11)
    sc = torch.exp(1.5 * torch.randn(1, Hkv, n, device="cuda", generator=g))     # heavy-tailed, like (a + eps) * ||v||
    sc = sc * torch.logspace(-0.5, 0.5, Hkv, device="cuda")[None, :, None]
    n_floor = ea.ea_n_floor(n_kept, 0.2)
    off = _check_against_oracle(ea, oracle, sc, n_kept, n_floor)
    sizes = np.diff(off[0])
    assert sizes.min() >= n_floor and sizes.max() > n_kept > sizes.min()


def test_adaptive_invalid_arguments(ea):
    sc = torch.rand(1, 2, 100, device="cuda")
    shape = ea.make_shape(1, 2, 2, 64, 100, 1)
    ctx = ea.Context.for_shape(shape)
    for n_kept, n_floor in [(101, 0), (-1, 0), (50, 51), (50, -1)]:
        with pytest.raises(ea.EAError) as e:
            ea.ea_select_compact_adaptive(ctx, shape, sc, n_kept, n_floor, gather=False)
        assert e.value.status == 1            # EA_ERR_INVALID_ARG
    small = ea.Context(0, 16)
    with pytest.raises(ea.EAError) as e:
        ea.ea_select_compact_adaptive(small, shape, sc, 10, 2, gather=False)
    assert e.value.status == 3                # EA_ERR_WORKSPACE
