"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's own formula: each compares an oracle
function with a library routine, a closed form, a sampling estimate, an
explicit per-position computation or brute-force enumeration.
"""
import itertools
import math

import numpy as np
import pytest
import torch

from paper_2510_00636_b200 import inputs


def bf16_bits(x):
    """float array -> (uint16 bit patterns after bf16 rounding, the rounded values as float64)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return inputs.bits(t), t.float().numpy().astype(np.float64)


def rotate(x, pos, base, layout="half"):
    """Rotary embedding written with complex numbers (independent of oracle and generator)."""
    d = x.shape[-1]
    m = np.arange(d // 2)
    theta = base ** (-2.0 * m / d)
    if layout == "half":
        z = x[..., : d // 2] + 1j * x[..., d // 2:]
    else:
        z = x[..., 0::2] + 1j * x[..., 1::2]
    z = z * np.exp(1j * pos * theta)
    out = np.empty_like(x)
    if layout == "half":
        out[..., : d // 2], out[..., d // 2:] = z.real, z.imag
    else:
        out[..., 0::2], out[..., 1::2] = z.real, z.imag
    return out


# ---------------------------------------------------------------- O1 mean / covariance
@pytest.mark.parametrize("norm", [0, 1])
def test_mean_cov_matches_numpy(oracle, norm):
    rng = np.random.default_rng(1)
    q_bits, q = bf16_bits(rng.normal(size=(3, 2, 40, 16)) * 3 + 1.5)
    mu, sigma = oracle.mean_cov(q_bits, cov_norm=norm)
    for u in range(3):
        for h in range(2):
            np.testing.assert_allclose(mu[u, h], q[u, h].mean(0), rtol=1e-13, atol=1e-13)
            ref = np.cov(q[u, h].T, bias=(norm == 0))
            np.testing.assert_allclose(sigma[u, h], ref, rtol=1e-11, atol=1e-12)
    # symmetric, positive semi-definite, rank at most W - 1
    q_bits, q = bf16_bits(rng.normal(size=(1, 1, 5, 12)))
    _, s = oracle.mean_cov(q_bits)
    s = s[0, 0]
    assert np.array_equal(s, s.T)
    ev = np.linalg.eigvalsh(s)
    assert ev.min() > -1e-12
    assert (ev > 1e-10).sum() <= 4


# ---------------------------------------------------------------- statistics from hidden states
@pytest.mark.parametrize("norm", [0, 1])
def test_hidden_statistics_equal_statistics_of_projected_samples(oracle, norm):
    """W_Q mu_h and W_Q Sigma_h W_Q^T against numpy's mean / cov of the explicitly projected rows."""
    rng = np.random.default_rng(31)
    U, W, dm, Hq, d = 4, 11, 24, 2, 8          # two weight sets, units set-major: 0, 0, 1, 1
    hb, h = bf16_bits(rng.normal(size=(U, W, dm)) + rng.normal(size=(U, 1, dm)))
    wb, wq = bf16_bits(rng.normal(size=(2, Hq * d, dm)) / np.sqrt(dm))
    mu, sigma = oracle.hidden_mean_cov(hb, wb, Hq, cov_norm=norm)
    for u in range(U):
        q = h[u] @ wq[u // 2].T                                    # [W, Hq*d]
        for j in range(Hq):
            qj = q[:, j * d:(j + 1) * d]
            np.testing.assert_allclose(mu[u, j], qj.mean(0), rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(sigma[u, j], np.cov(qj.T, bias=(norm == 0)), rtol=1e-10, atol=1e-13)


def test_hidden_statistics_with_selector_projection_are_window_statistics(oracle):
    """W_Q that picks d hidden channels per head: the result is mean_cov of those channels."""
    rng = np.random.default_rng(32)
    U, W, Hq, d = 2, 9, 3, 4
    dm = Hq * d
    hb, _ = bf16_bits(rng.normal(size=(U, W, dm)))
    wb, _ = bf16_bits(np.eye(dm)[None])
    mu, sigma = oracle.hidden_mean_cov(hb, wb, Hq)
    q_win = hb.reshape(U, W, Hq, d).transpose(0, 2, 1, 3)           # [U, Hq, W, d]
    mu2, sigma2 = oracle.mean_cov(q_win)
    np.testing.assert_allclose(mu, mu2, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(sigma, sigma2, rtol=1e-12, atol=1e-15)
    # scaling the projection by c scales the mean by c and the covariance by c^2
    wb2, _ = bf16_bits(2.0 * np.eye(dm)[None])
    mu3, sigma3 = oracle.hidden_mean_cov(hb, wb2, Hq)
    np.testing.assert_allclose(mu3, 2.0 * mu, rtol=1e-13)
    np.testing.assert_allclose(sigma3, 4.0 * sigma, rtol=1e-13)
    # and the whole statistics step agrees with the window form
    pos = np.array([7, 100], np.int64)
    a = oracle.query_stats_hidden(hb, wb, Hq, pos, 5, 1e4)
    b = oracle.query_stats(q_win, pos, 5, 1e4)
    np.testing.assert_allclose(a[0], b[0], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(a[1], b[1], rtol=1e-12, atol=1e-15)


# ---------------------------------------------------------------- O2 averaged rotation
@pytest.mark.parametrize("pos,T,base,d", [(512, 512, 1e4, 64), (8192, 512, 5e5, 128),
                                          (131072, 1024, 1e6, 256), (0, 1, 1e4, 8), (7, 3, 10.0, 4)])
def test_rope_average_closed_form(oracle, pos, T, base, d):
    """Geometric series: (1/T) sum_j e^{i theta (p+j)} = e^{i theta (p+(T-1)/2)} sin(T theta/2) / (T sin(theta/2))."""
    cbar, sbar = oracle.rope_average(np.array([pos]), T, base, d)
    theta = base ** (-2.0 * np.arange(d // 2) / d)
    z = np.exp(1j * theta * (pos + (T - 1) / 2)) * np.sin(T * theta / 2) / (T * np.sin(theta / 2))
    np.testing.assert_allclose(cbar[0], z.real, rtol=0, atol=1e-11)
    np.testing.assert_allclose(sbar[0], z.imag, rtol=0, atol=1e-11)
    assert np.all(cbar ** 2 + sbar ** 2 <= 1 + 1e-12)


def test_rope_average_special_cases(oracle):
    # T = 1: the average is the rotation at pos_next itself (orthogonal blocks)
    cbar, sbar = oracle.rope_average(np.array([37]), 1, 1e4, 16)
    np.testing.assert_allclose(cbar ** 2 + sbar ** 2, 1.0, atol=1e-14)
    theta = 1e4 ** (-2.0 * np.arange(8) / 16)
    np.testing.assert_allclose(cbar[0], np.cos(37 * theta), atol=1e-14)
    np.testing.assert_allclose(sbar[0], np.sin(37 * theta), atol=1e-14)
    # channel 0 has theta = 1: the average over many positions nearly cancels
    cbar, sbar = oracle.rope_average(np.array([100]), 512, 1e4, 16)
    assert math.hypot(cbar[0, 0], sbar[0, 0]) < 5e-3
    # huge base: the slow channels barely rotate, their block stays close to the identity
    cbar, sbar = oracle.rope_average(np.array([0]), 4, 1e30, 8)
    np.testing.assert_allclose(cbar[0, 1:], 1.0, atol=1e-6)
    np.testing.assert_allclose(sbar[0, 1:], 0.0, atol=1e-6)
    # several units at once
    c2, s2 = oracle.rope_average(np.array([5, 900]), 16, 1e4, 8)
    c5, _ = oracle.rope_average(np.array([5]), 16, 1e4, 8)
    c9, _ = oracle.rope_average(np.array([900]), 16, 1e4, 8)
    assert np.array_equal(c2[0], c5[0]) and np.array_equal(c2[1], c9[0])


# ---------------------------------------------------------------- O3 averaged Gaussian
@pytest.mark.parametrize("layout", ["half", "interleaved"])
def test_averaged_gaussian_equals_statistics_of_rotated_samples(oracle, layout):
    """mu_bar / Sigma_bar must be the mean / covariance of the window queries after each is
    rotated to every future position and averaged over positions (explicit, sample by sample)."""
    rng = np.random.default_rng(2)
    U, Hq, W, d, T, base = 2, 3, 24, 16, 11, 50.0
    pos = np.array([40, 3])
    q_bits, q = bf16_bits(rng.normal(size=(U, Hq, W, d)) + 0.7)
    lay = 0 if layout == "half" else 1
    mu_bar, sigma_bar = oracle.query_stats(q_bits, pos, T, base, layout=lay)
    for u in range(U):
        qbar = np.mean([rotate(q[u], pos[u] + j, base, layout) for j in range(T)], axis=0)
        for h in range(Hq):
            np.testing.assert_allclose(mu_bar[u, h], qbar[h].mean(0), atol=1e-12)
            np.testing.assert_allclose(sigma_bar[u, h], np.cov(qbar[h].T, bias=True), atol=1e-12)


def test_rotation_convention_matches_key_generator(oracle):
    """The generator's rotary embedding of keys and the oracle's averaged rotation of queries
    use one convention: mean_j (R_{p+j} q) . (R_i k) equals (R_bar q) . (R_i k), and the
    generator's rotation gives scores that depend on relative position only."""
    rng = np.random.default_rng(3)
    d, base, T, p = 32, 1e3, 9, 77
    q = rng.normal(size=(1, d))
    k = rng.normal(size=(1, d))
    kt = lambda pos: inputs.rope_half_split(torch.tensor(k, dtype=torch.float32),
                                            torch.tensor([pos]), base).double().numpy()
    qt = lambda pos: inputs.rope_half_split(torch.tensor(q, dtype=torch.float32),
                                            torch.tensor([pos]), base).double().numpy()
    # relative-position property of the generator's embedding
    assert abs((qt(50) @ kt(20).T).item() - (qt(130) @ kt(100).T).item()) < 1e-4
    np.testing.assert_allclose(kt(20), rotate(k.astype(np.float32).astype(np.float64), 20, base), atol=1e-5)
    # oracle's R_bar applied to a single "mean" vector with zero covariance
    cbar, sbar = oracle.rope_average(np.array([p]), T, base, d)
    mu_bar, sig_bar = oracle.apply_rope_average(q.reshape(1, 1, d), np.zeros((1, 1, d, d)), cbar, sbar)
    want = np.mean([(rotate(q, p + j, base) @ rotate(k, 5, base).T).item() for j in range(T)])
    got = (mu_bar[0, 0] @ rotate(k, 5, base).T).item()
    assert abs(want - got) < 1e-12
    assert np.all(sig_bar == 0)


# ---------------------------------------------------------------- O4 closed-form expectation
def _small_problem(rng, U=1, Hq=2, Hkv=1, W=32, d=8, n=12, qscale=0.6):
    q_bits, q = bf16_bits(rng.normal(size=(U, Hq, W, d)) * qscale + 0.2)
    k_bits, k = bf16_bits(rng.normal(size=(U, Hkv, n, d)))
    v_bits, v = bf16_bits(rng.normal(size=(U, Hkv, n, d)))
    return q_bits, q, k_bits, k, v_bits, v


def test_logits_match_monte_carlo_expectation(oracle):
    """exp(s_i) must equal E[exp(q.k_i/sqrt(d))] for q ~ N(mu_bar, Sigma_bar) (Gaussian MGF)."""
    rng = np.random.default_rng(4)
    d, n = 8, 12
    q_bits, q, k_bits, k, _, _ = _small_problem(rng, d=d, n=n)
    mu_bar, sigma_bar = oracle.query_stats(q_bits, np.array([20]), 6, 100.0)
    s = oracle.logits(k_bits, mu_bar, sigma_bar)
    N = 400_000
    for h in range(2):
        w, V = np.linalg.eigh(sigma_bar[0, h])
        L = V * np.sqrt(np.clip(w, 0, None))
        samples = mu_bar[0, h] + rng.normal(size=(N, d)) @ L.T
        e = np.exp(samples @ k[0, 0].T / math.sqrt(d))           # [N, n]
        est, se = e.mean(0), e.std(0, ddof=1) / math.sqrt(N)
        z = (est - np.exp(s[0, h])) / se
        assert np.all(np.abs(z) < 4.5), z
        # the quadratic term matters here: the estimate excludes the mean-only formula
        lin_only = np.exp(k[0, 0] @ mu_bar[0, h] / math.sqrt(d))
        assert np.any(np.abs(est - lin_only) / se > 10)


def test_logits_zero_covariance_is_dot_product(oracle):
    """All window queries equal => Sigma = 0 and s_i = (R_bar u) . k_i / sqrt(d)."""
    rng = np.random.default_rng(5)
    d, n, W, T, base, p = 16, 20, 10, 7, 1e3, 31
    u_bits, u = bf16_bits(rng.normal(size=(d,)))
    q_bits = np.broadcast_to(u_bits, (1, 1, W, d)).copy()
    k_bits, k = bf16_bits(rng.normal(size=(1, 1, n, d)))
    mu_bar, sigma_bar = oracle.query_stats(q_bits, np.array([p]), T, base)
    assert np.abs(sigma_bar).max() < 1e-28
    s = oracle.logits(k_bits, mu_bar, sigma_bar)
    ubar = np.mean([rotate(u, p + j, base) for j in range(T)], axis=0)
    np.testing.assert_allclose(s[0, 0], k[0, 0] @ ubar / math.sqrt(d), atol=1e-12)


def test_logits_equal_mean_and_variance_of_projected_window(oracle):
    """s_i = mean_w(k_i.qbar_w)/sqrt(d) + var_w(k_i.qbar_w)/(2d), qbar_w the averaged-rotated samples."""
    rng = np.random.default_rng(6)
    U, Hq, Hkv, W, d, n, T, base = 2, 4, 2, 20, 16, 33, 5, 200.0
    pos = np.array([33, 64])
    q_bits, q, k_bits, k, _, _ = _small_problem(rng, U, Hq, Hkv, W, d, n, qscale=2.0)
    mu_bar, sigma_bar = oracle.query_stats(q_bits, pos, T, base)
    s = oracle.logits(k_bits, mu_bar, sigma_bar)
    for u in range(U):
        qbar = np.mean([rotate(q[u], pos[u] + j, base) for j in range(T)], axis=0)   # [Hq, W, d]
        for h in range(Hq):
            proj = k[u, h // 2] @ qbar[h].T                                            # [n, W]
            want = proj.mean(1) / math.sqrt(d) + proj.var(1) / (2 * d)
            np.testing.assert_allclose(s[u, h], want, rtol=1e-11, atol=1e-11)


# ---------------------------------------------------------------- O5-O7 softmax, GQA, value norm
def test_scores_invariants(oracle):
    rng = np.random.default_rng(7)
    U, Hq, Hkv, n, d = 2, 6, 2, 50, 8
    s = rng.normal(size=(U, Hq, n)) * 4
    v_bits, v = bf16_bits(rng.normal(size=(U, Hkv, n, d)))
    vnorm = np.linalg.norm(v, axis=-1)
    sc, a = oracle.scores(s, v_bits, 0.02, oracle.GROUP_MEAN_PROB, return_attention=True)
    np.testing.assert_allclose(a.sum(-1), 1.0, atol=1e-13)
    np.testing.assert_allclose(sc, (a + 0.02) * vnorm, rtol=1e-13)
    # scipy's softmax as the library routine for Eq. 8
    from scipy.special import softmax
    ref = softmax(s, axis=-1).reshape(U, Hkv, 3, n).mean(2)
    np.testing.assert_allclose(a, ref, rtol=1e-12, atol=1e-15)
    _, a_sum = oracle.scores(s, v_bits, 0.0, oracle.GROUP_SUM_PROB, return_attention=True)
    np.testing.assert_allclose(a_sum, 3 * ref, rtol=1e-12, atol=1e-15)
    _, a_ml = oracle.scores(s, v_bits, 0.0, oracle.GROUP_MEAN_LOGIT, return_attention=True)
    np.testing.assert_allclose(a_ml, softmax(s.reshape(U, Hkv, 3, n).mean(2), axis=-1), rtol=1e-12)
    # adding a per-head constant to the logits changes nothing, even a huge one
    shift = rng.normal(size=(U, Hq, 1)) * 1e5
    sc2 = oracle.scores(s + shift, v_bits, 0.02)
    np.testing.assert_allclose(sc2, sc, rtol=1e-9)
    # logits far beyond exp's range stay finite
    big = oracle.scores(s * 1e4, v_bits, 0.02)
    assert np.all(np.isfinite(big))
    # scaling V by c scales the scores by c and keeps the kept set
    v2_bits, _ = bf16_bits(v * 4.0)
    sc4 = oracle.scores(s, v2_bits, 0.02)
    np.testing.assert_allclose(sc4, 4 * sc, rtol=1e-13)
    assert np.array_equal(oracle.select(sc4, 17), oracle.select(sc, 17))


def test_group_modes_coincide_without_grouping(oracle):
    rng = np.random.default_rng(8)
    s = rng.normal(size=(1, 3, 30)) * 3
    v_bits, _ = bf16_bits(rng.normal(size=(1, 3, 30, 4)))
    base = oracle.scores(s, v_bits, 0.02, oracle.GROUP_MEAN_PROB)
    for mode in (oracle.GROUP_SUM_PROB, oracle.GROUP_MEAN_LOGIT):
        np.testing.assert_allclose(oracle.scores(s, v_bits, 0.02, mode), base, rtol=1e-13)


# ---------------------------------------------------------------- Eq. 9 with the output projection
def test_scores_with_output_projection(oracle):
    rng = np.random.default_rng(41)
    U, Hq, Hkv, n, d, dm = 2, 4, 2, 13, 8, 12
    G = Hq // Hkv
    s = rng.normal(size=(U, Hq, n)) * 3
    vb, v = bf16_bits(rng.normal(size=(U, Hkv, n, d)))
    wb, wo = bf16_bits(rng.normal(size=(2, dm, Hq * d)))
    for mode in (0, 1):
        got = oracle.scores_wo(s, vb, wb, 0.02, group_mode=mode)
        # numpy restatement through the softmax library form and explicit matrix-vector products
        a_hat = np.exp(s - s.max(-1, keepdims=True))
        a_hat /= a_hat.sum(-1, keepdims=True)
        want = np.zeros((U, Hkv, n))
        for u in range(U):
            for h in range(Hq):
                g = h // G
                y = v[u, g] @ wo[u][:, h * d:(h + 1) * d].T              # [n, dm]; one set per unit
                want[u, g] += (a_hat[u, h] + 0.02) * np.linalg.norm(y, axis=-1)
        if mode == 0:
            want /= G
        np.testing.assert_allclose(got, want, rtol=1e-12)
    # an output projection with orthonormal columns per head leaves the norm of v unchanged:
    # the score falls back to the ||v|| form
    q, _ = np.linalg.qr(rng.normal(size=(dm, d)))                          # [dm, d], orthonormal columns
    wo_iso = np.concatenate([q] * Hq, axis=1)[None]
    wb_iso, wo_iso_r = bf16_bits(wo_iso)
    got = oracle.scores_wo(s, vb, wb_iso, 0.02)
    plain = oracle.scores(s, vb, 0.02)
    np.testing.assert_allclose(got, plain, rtol=2e-2)                      # bf16 rounding of the projection
    # exactly so for a selector matrix (representable in bf16)
    sel = np.zeros((dm, d)); sel[:d, :d] = np.eye(d)
    wb_sel, _ = bf16_bits(np.concatenate([sel] * Hq, axis=1)[None])
    np.testing.assert_allclose(oracle.scores_wo(s, vb, wb_sel, 0.02), plain, rtol=1e-12)
    np.testing.assert_allclose(oracle.scores_wo(s, vb, wb_sel, 0.0, group_mode=1),
                               oracle.scores(s, vb, 0.0, group_mode=1), rtol=1e-12)
    with pytest.raises(ValueError):
        oracle.scores_wo(s, vb, wb_sel, 0.02, group_mode=2)


# ---------------------------------------------------------------- O8-O9 selection and compaction
def test_select_brute_force(oracle):
    rng = np.random.default_rng(9)
    for n, kept in [(1, 1), (6, 0), (9, 4), (12, 12), (13, 5)]:
        sc = rng.random(size=(3, n))
        idx = oracle.select(sc, kept)
        assert idx.shape == (3, kept)
        for h in range(3):
            best = max(itertools.combinations(range(n), kept), key=lambda c: sc[h, list(c)].sum())
            assert list(idx[h]) == sorted(best)


def test_select_ties_take_lowest_index(oracle):
    sc = np.array([[1.0, 3.0, 3.0, 0.5, 3.0, 3.0, 2.0, 3.0]])
    assert list(oracle.select(sc, 3)[0]) == [1, 2, 4]
    assert list(oracle.select(sc, 6)[0]) == [1, 2, 4, 5, 6, 7]
    assert list(oracle.select(np.zeros((1, 7)), 4)[0]) == [0, 1, 2, 3]
    # every subset of the same total is valid; the rule picks the lexicographically first
    n, kept = 10, 4
    sc = np.array([[2.0, 1, 2, 1, 2, 1, 1, 2, 1, 1]])
    best_sum = max(sc[0, list(c)].sum() for c in itertools.combinations(range(n), kept))
    ties = [c for c in itertools.combinations(range(n), kept) if sc[0, list(c)].sum() == best_sum]
    assert list(oracle.select(sc, kept)[0]) == list(min(ties))


def test_select_follows_permutation(oracle):
    rng = np.random.default_rng(10)
    sc = rng.random(size=(2, 40))
    perm = rng.permutation(40)
    a = oracle.select(sc, 11)
    b = oracle.select(sc[:, perm], 11)
    for h in range(2):
        assert sorted(perm[b[h]]) == list(a[h])


def test_gather(oracle):
    rng = np.random.default_rng(11)
    rows = rng.integers(0, 65535, size=(2, 3, 9, 4), dtype=np.uint16)
    idx = np.sort(rng.permuted(np.tile(np.arange(9), (2, 3, 1)), axis=-1)[..., :5], axis=-1).astype(np.int32)
    out = oracle.gather(rows, idx)
    assert np.array_equal(out, np.take_along_axis(rows, idx[..., None].astype(np.int64), axis=2))


# ---------------------------------------------------------------- head-adaptive selection
def _per_head(idx, off, u):
    return [list(idx[u, off[u, g]:off[u, g + 1]]) for g in range(off.shape[1] - 1)]


def test_adaptive_select_brute_force(oracle):
    """The kept set maximises the total score over all sets of the unit's budget that hold at least
    n_floor keys of every head (distinct scores: the maximiser is unique)."""
    rng = np.random.default_rng(21)
    for Hkv, n, kept, floor in [(2, 5, 2, 1), (2, 5, 3, 0), (3, 4, 2, 1), (2, 6, 3, 3), (3, 4, 1, 0), (2, 6, 4, 2)]:
        sc = rng.random(size=(2, Hkv, n))
        idx, off = oracle.select_adaptive(sc, kept, floor)
        B = Hkv * kept
        assert idx.shape == (2, B) and off.shape == (2, Hkv + 1)
        for u in range(2):
            flat = sc[u].reshape(-1)
            best, best_sum = None, -1.0
            for c in itertools.combinations(range(Hkv * n), B):
                per_head = np.bincount(np.asarray(c) // n, minlength=Hkv)
                if per_head.min() < floor:
                    continue
                tot = flat[list(c)].sum()
                if tot > best_sum:
                    best, best_sum = c, tot
            got = [g * n + i for g, lst in enumerate(_per_head(idx, off, u)) for i in lst]
            assert got == sorted(best)
            assert off[u, 0] == 0 and off[u, -1] == B


def test_adaptive_select_limits_reduce_to_library_routines(oracle):
    rng = np.random.default_rng(22)
    U, Hkv, n, kept = 3, 4, 50, 13
    sc = rng.random(size=(U, Hkv, n))
    # safeguard = whole budget: plain per-head selection
    idx, off = oracle.select_adaptive(sc, kept, kept)
    assert np.array_equal(off, np.tile(np.arange(Hkv + 1) * kept, (U, 1)))
    assert np.array_equal(idx.reshape(U, Hkv, kept), oracle.select(sc, kept))
    # no safeguard: the Hkv * kept largest of the flattened unit (numpy's sort as the library routine)
    idx, off = oracle.select_adaptive(sc, kept, 0)
    for u in range(U):
        top = np.sort(np.argsort(-sc[u].reshape(-1), kind="stable")[: Hkv * kept])
        got = [g * n + i for g, lst in enumerate(_per_head(idx, off, u)) for i in lst]
        assert got == list(top)


def test_adaptive_select_ties_go_to_the_lower_head_then_index(oracle):
    # all scores equal: the safeguard takes the first n_floor keys of every head, the other places go
    # to head 0 until it is full, then head 1, ...
    Hkv, n, kept, floor = 3, 6, 3, 1
    idx, off = oracle.select_adaptive(np.ones((1, Hkv, n)), kept, floor)
    assert _per_head(idx, off, 0) == [[0, 1, 2, 3, 4, 5], [0, 1], [0]]
    # one tie across heads at the threshold
    sc = np.array([[[5.0, 1.0, 3.0, 0.0], [4.0, 3.0, 0.5, 3.0]]])
    idx, off = oracle.select_adaptive(sc, 2, 1)           # budget 4: 5, 4 (safeguards), then 3 (head 0), 3 (head 1, idx 1)
    assert _per_head(idx, off, 0) == [[0, 2], [0, 1]]
    idx, off = oracle.select_adaptive(sc, 2, 0)           # no safeguard: 5, 4, 3 (head 0), 3 (head 1, idx 1)
    assert _per_head(idx, off, 0) == [[0, 2], [0, 1]]


def test_adaptive_select_invariants(oracle):
    rng = np.random.default_rng(23)
    U, Hkv, n, kept, floor = 2, 4, 200, 30, 10
    plain = rng.random(size=(U, Hkv, n))
    skewed = plain.copy()
    skewed[:, 1] *= 10.0                                 # one head matters far more than the others
    for sc in (plain, skewed):
        idx, off = oracle.select_adaptive(sc, kept, floor)
        for u in range(U):
            heads = _per_head(idx, off, u)
            sizes = [len(h) for h in heads]
            assert sum(sizes) == Hkv * kept and min(sizes) >= floor
            if sc is skewed:
                # about 170 keys of the strong head beat every key of the others: it takes every free place
                assert sizes == [floor, floor + Hkv * (kept - floor), floor, floor]
            else:
                assert max(sizes) > kept > min(sizes)     # the budget really moves between heads
            beyond_floor_min, dropped_max = np.inf, -np.inf
            for g, lst in enumerate(heads):
                assert lst == sorted(set(lst))
                # within a head the kept keys are its best ones
                assert lst == list(oracle.select(sc[u, g][None], len(lst))[0])
                order = np.sort(sc[u, g])[::-1]
                if len(lst) > floor:
                    beyond_floor_min = min(beyond_floor_min, order[len(lst) - 1])
                if len(lst) < n:
                    dropped_max = max(dropped_max, order[max(len(lst), floor)])
            # one threshold for the whole unit separates what was kept beyond the safeguard from what was dropped
            assert beyond_floor_min >= dropped_max
        # scaling every score of the unit by a positive constant changes nothing
        idx2, off2 = oracle.select_adaptive(sc * 3.0, kept, floor)
        assert np.array_equal(idx, idx2) and np.array_equal(off, off2)


def test_adaptive_gather_and_floor(oracle):
    rng = np.random.default_rng(24)
    U, Hkv, n, d, kept, floor = 2, 3, 9, 4, 4, 1
    rows = rng.integers(0, 65535, size=(U, Hkv, n, d), dtype=np.uint16)
    sc = rng.random(size=(U, Hkv, n))
    idx, off = oracle.select_adaptive(sc, kept, floor)
    out = oracle.gather_adaptive(rows, idx, off)
    for u in range(U):
        want = np.concatenate([rows[u, g][lst] for g, lst in enumerate(_per_head(idx, off, u))])
        assert np.array_equal(out[u], want)
    assert oracle.n_floor(4096, 0.2) == 819 and oracle.n_floor(256, 0.2) == 51
    assert oracle.n_floor(10, 0.0) == 0 and oracle.n_floor(10, 1.0) == 10


def test_n_kept_is_truncated_product(oracle):
    assert oracle.n_kept(512, 0.5) == 256
    assert oracle.n_kept(8192, 0.5) == 4096
    assert oracle.n_kept(32768, 0.75) == 8192
    assert oracle.n_kept(131072, 0.875) == 16384
    assert oracle.n_kept(10, 0.0) == 10 and oracle.n_kept(10, 1.0) == 0
    rng = np.random.default_rng(12)
    for _ in range(200):
        n, r = int(rng.integers(0, 10**6)), float(rng.random())
        assert oracle.n_kept(n, r) == int(n * (1 - r))


# ---------------------------------------------------------------- whole path
def test_whole_path_single_head_against_array_formulation(oracle):
    """One head, eps = 0: the compression routine written with whole-array library operations
    (matrix products, softmax, norms, a stable descending sort) selects the same pairs."""
    from scipy.special import softmax
    rng = np.random.default_rng(13)
    W, d, n, T, base, kept = 48, 16, 200, 8, 1e3, 60
    q_bits, q = bf16_bits(rng.normal(size=(1, 1, W, d)) * 1.5 + 0.3)
    k_bits, k = bf16_bits(rng.normal(size=(1, 1, n, d)))
    v_bits, v = bf16_bits(rng.normal(size=(1, 1, n, d)) * np.exp(0.5 * rng.normal(size=(1, 1, n, 1))))
    out = oracle.compress(q_bits, k_bits, v_bits, np.array([n]), T, base, 0.0, kept)
    qbar = np.mean([rotate(q[0, 0], n + j, base) for j in range(T)], axis=0)
    mean_query, cov_query = qbar.mean(0), np.cov(qbar.T, bias=True)
    keys, values = k[0, 0], v[0, 0]
    sc = keys @ mean_query / math.sqrt(d) + np.einsum("ni,ij,nj->n", keys, cov_query, keys) / (2 * d)
    sc = softmax(sc) * np.linalg.norm(values, axis=-1)
    top = np.sort(np.argsort(-sc, kind="stable")[:kept])
    assert np.array_equal(out["kept_idx"][0, 0], top)
    np.testing.assert_allclose(out["scores"][0, 0], sc, rtol=1e-10)
    assert np.array_equal(out["k_out"][0, 0], k_bits[0, 0][top])
    assert np.array_equal(out["v_out"][0, 0], v_bits[0, 0][top])


def test_oracle_on_tiny_config(oracle):
    """Config 0 end to end: shapes, finiteness, and the one-hot character of its softmax."""
    cfg = inputs.CONFIGS[0]
    q, k, v, pos = inputs.generate_layer(cfg)
    out = oracle.compress(inputs.bits(q), inputs.bits(k), inputs.bits(v), pos.numpy(), cfg.n_future,
                          cfg.rope_base, cfg.eps, cfg.n_kept)
    assert out["kept_idx"].shape == (1, 2, 256)
    assert np.all(np.isfinite(out["logits"])) and np.all(np.isfinite(out["scores"]))
    assert np.all(np.diff(out["kept_idx"], axis=-1) > 0)


# ------------------------------------------------------------------------------------------
# Streaming driver (oracle/ea_stream.py): plumbing around the pinned functions.
def _stream_inputs(seed, U=1, Hq=4, Hkv=2, d=64, n0=40, W=16):
    rng = np.random.default_rng(seed)
    def bf(x):
        return (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    k0, v0 = bf(rng.normal(size=(U, Hkv, n0, d))), bf(rng.normal(size=(U, Hkv, n0, d)))
    return rng, bf, k0, v0


def test_stream_single_event_is_compress_on_the_concatenated_inputs(oracle):
    from oracle.ea_stream import StreamOracle
    rng, bf, k0, v0 = _stream_inputs(1)
    k1, v1 = bf(rng.normal(size=(1, 2, 24, 64))), bf(rng.normal(size=(1, 2, 24, 64)))
    q = bf(rng.normal(size=(1, 4, 16, 64)) + 0.3)
    st = StreamOracle(k0, v0, window=16, budget=32)
    st.append(k1, v1)
    st.push_queries(q)
    got = st.compress([64], 8, 1e4, 0.02)
    want = oracle.compress(q, np.concatenate([k0, k1], 2), np.concatenate([v0, v1], 2), np.array([64]), 8, 1e4,
                           0.02, 32)
    assert np.array_equal(got["kept_idx"], want["kept_idx"])
    assert np.array_equal(got["scores"], want["scores"])
    st.keep(got["kept_idx"])
    assert st.n_keys == 32 and np.array_equal(st.k, want["k_out"]) and np.array_equal(st.v, want["v_out"])


def test_stream_window_is_the_tail_of_everything_pushed(oracle):
    from oracle.ea_stream import StreamOracle
    rng, bf, k0, v0 = _stream_inputs(2)
    st = StreamOracle(k0, v0, window=16, budget=1000)
    pushed = []
    for m in (5, 7, 3, 20, 1, 40):          # partly filled, exactly full, wrapped several times in one push
        q = bf(rng.normal(size=(1, 4, m, 64)))
        pushed.append(q)
        st.push_queries(q)
        everything = np.concatenate(pushed, axis=2)
        assert np.array_equal(st.q, everything[:, :, -16:])
        assert st.q.shape[2] == min(16, everything.shape[2])
    # statistics depend on the set of rows only: any rotation of the window gives the same mean and covariance
    mu, sig = oracle.mean_cov(st.q)
    mu_r, sig_r = oracle.mean_cov(np.roll(st.q, 5, axis=2))
    np.testing.assert_allclose(mu, mu_r, rtol=0, atol=1e-15)
    np.testing.assert_allclose(sig, sig_r, rtol=0, atol=1e-14)


def test_stream_events_compose_as_index_maps(oracle):
    """After two events the cache holds original rows: following the kept indices back through both events
    names them, and below the budget an event keeps every row."""
    from oracle.ea_stream import StreamOracle
    rng, bf, k0, v0 = _stream_inputs(3, n0=20)
    st = StreamOracle(k0, v0, window=16, budget=48)
    origin = np.broadcast_to(np.arange(20), (1, 2, 20)).copy()       # which original row sits where
    all_k = k0
    for e, n_new in enumerate((12, 30, 30)):
        k1, v1 = bf(rng.normal(size=(1, 2, n_new, 64))), bf(rng.normal(size=(1, 2, n_new, 64)))
        st.append(k1, v1)
        st.push_queries(bf(rng.normal(size=(1, 4, 9, 64)) + 0.1 * e))
        origin = np.concatenate([origin, np.broadcast_to(np.arange(all_k.shape[2], all_k.shape[2] + n_new),
                                                         (1, 2, n_new))], axis=2)
        all_k = np.concatenate([all_k, k1], axis=2)
        out = st.compress([all_k.shape[2]], 8, 1e4, 0.02)
        idx = out["kept_idx"]
        if e == 0:
            assert st.n_keys == 32 and np.array_equal(idx, np.broadcast_to(np.arange(32), (1, 2, 32)))
        assert idx.shape[2] == min(st.n_keys, 48)
        assert (np.diff(idx, axis=2) > 0).all()
        st.keep(idx)
        origin = np.take_along_axis(origin, idx.astype(np.int64), axis=2)
        for g in range(2):
            assert np.array_equal(st.k[0, g], all_k[0, g][origin[0, g]])


# ------------------------------------------------------------------------------------------
# Quantised cache (oracle/ea_quant.py)
def test_e4m3_decoder_against_a_library_conversion_of_every_code():
    """All 256 codes: the formula of the format against torch's float8_e4m3fn -> float32 conversion."""
    import torch
    from oracle import ea_quant
    codes = np.arange(256, dtype=np.uint8)
    want = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    got = ea_quant.e4m3_decode(codes)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.isnan(got).sum() == 2
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    assert got[ok].max() == 448.0 and np.abs(got[ok][got[ok] != 0]).min() == 2.0 ** -9
    # and back: every finite value re-encodes to its own code (up to the sign of zero)
    back = torch.from_numpy(got[ok].astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(back, codes[ok])


def _quant_case(seed, U=2, Hq=4, Hkv=2, d=64, n=96, W=24):
    import torch
    rng = np.random.default_rng(seed)
    def bf(x):
        return (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    q = bf(rng.normal(size=(U, Hq, W, d)) * 0.7 + 0.2)
    k = rng.normal(size=(U, Hkv, n, d)) * (1 + 3 * (rng.random(d) < 0.05))
    v = rng.normal(size=(U, Hkv, n, d)) * np.exp(0.5 * rng.normal(size=(U, Hkv, n, 1)))
    k_scale = (np.abs(k).max(2) / 448.0).astype(np.float32)                  # per channel
    v_scale = (np.abs(v).max(3) / 448.0).astype(np.float32)                  # per token
    enc = lambda x: torch.from_numpy(x.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    return q, enc(k / k_scale[:, :, None, :]), k_scale, enc(v / v_scale[..., None]), v_scale


def test_quantised_scoring_equals_scoring_with_the_key_scales_folded_into_the_statistics(oracle):
    """k = diag(s) k_q, so mu.k = (s*mu).k_q and k^T Sigma k = k_q^T (diag(s) Sigma diag(s)) k_q: an exact
    identity, which is also how a kernel can consume the codes without ever forming the scaled keys."""
    from oracle import ea_quant
    q, kq, ks, vq, vs = _quant_case(11)
    pos = np.array([96, 200])
    mu, sig = oracle.query_stats(q, pos, 16, 1e4)
    direct = ea_quant.logits(ea_quant.dequant_k(kq, ks), mu, sig)
    G = mu.shape[1] // kq.shape[1]
    s_q = np.repeat(ks.astype(np.float64), G, axis=1)                       # [U, Hq, d]
    folded = ea_quant.logits(ea_quant.e4m3_decode(kq), mu * s_q, sig * s_q[..., :, None] * s_q[..., None, :])
    np.testing.assert_allclose(folded, direct, rtol=1e-12, atol=1e-12)
    # value side: ||s_i v_q|| = s_i ||v_q||
    sc = ea_quant.scores(direct, ea_quant.dequant_v(vq, vs), 0.02)
    unit = ea_quant.scores(direct, ea_quant.e4m3_decode(vq), 0.0) * vs
    sc0 = ea_quant.scores(direct, ea_quant.dequant_v(vq, vs), 0.0)
    np.testing.assert_allclose(unit, sc0, rtol=1e-12)
    assert (sc > sc0).all()


def test_quantised_oracle_with_unit_scales_is_the_bf16_oracle(oracle):
    """E4M3 values are bf16 values: with all scales one, the quantised path must reproduce the pinned C oracle
    run on the same numbers as bf16 bits, through every step including the kept rows."""
    from oracle import ea_quant
    q, kq, ks, vq, vs = _quant_case(12)
    ks[:], vs[:] = 1.0, 1.0
    to_bf16 = lambda codes: (ea_quant.e4m3_decode(codes).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    pos = np.array([96, 96])
    got = ea_quant.compress(q, kq, ks, vq, vs, pos, 16, 1e4, 0.02, 40)
    want = oracle.compress(q, to_bf16(kq), to_bf16(vq), pos, 16, 1e4, 0.02, 40)
    np.testing.assert_allclose(got["logits"], want["logits"], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(got["scores"], want["scores"], rtol=1e-11)
    assert np.array_equal(got["kept_idx"], want["kept_idx"])
    assert np.array_equal(to_bf16(got["k_out"]), want["k_out"]) and np.array_equal(to_bf16(got["v_out"]), want["v_out"])
    for mode in (1, 2):
        s = got["logits"]
        np.testing.assert_allclose(ea_quant.scores(s, ea_quant.e4m3_decode(vq), 0.02, mode),
                                   oracle.scores(s, to_bf16(vq), 0.02, group_mode=mode), rtol=1e-11)


def test_fill_holes_is_a_permutation_of_the_kept_set_that_moves_only_the_tail(oracle):
    """The unordered compaction map: same kept set, rows below n_kept that are kept do not move, exactly the
    kept rows beyond n_kept move, and they fill the evicted positions in ascending order of both; checked
    on every subset of a small cache by brute force."""
    from itertools import combinations
    from oracle.ea_stream import fill_holes
    n, n_kept = 7, 4
    for kept in combinations(range(n), n_kept):
        where = fill_holes(np.array([kept], dtype=np.int32), n_kept)[0]
        assert sorted(where) == list(kept)
        for p in range(n_kept):
            if p in kept:
                assert where[p] == p
        moved_to = [p for p in range(n_kept) if where[p] != p]
        assert [where[p] for p in moved_to] == [i for i in kept if i >= n_kept]
        assert moved_to == [p for p in range(n_kept) if p not in kept]
    rng = np.random.default_rng(0)
    sc = rng.random((2, 3, 50))
    idx = oracle.select(sc, 20)
    where = fill_holes(idx, 20)
    assert np.array_equal(np.sort(where, axis=-1), idx)
    ident = fill_holes(np.broadcast_to(np.arange(20, dtype=np.int32), (2, 3, 20)), 20)
    assert np.array_equal(ident, np.broadcast_to(np.arange(20), (2, 3, 20)))


# ------------------------------------------------------------------------------------------
# Streaming on a quantised cache (oracle/ea_stream.py, QuantStreamOracle)
def test_quantised_stream_single_event_is_quantised_compress_on_the_concatenated_inputs(oracle):
    from oracle import ea_quant
    from oracle.ea_stream import QuantStreamOracle
    q, kq, ks, vq, vs = _quant_case(21, U=1, n=96, W=16)
    st = QuantStreamOracle(kq[:, :, :60], ks, vq[:, :, :60], vs[:, :, :60], window=16, budget=50)
    st.append(kq[:, :, 60:], vq[:, :, 60:], vs[:, :, 60:])
    st.push_queries(q)
    got = st.compress([96], 8, 1e4, 0.02)
    want = ea_quant.compress(q, kq, ks, vq, vs, np.array([96]), 8, 1e4, 0.02, 50)
    assert np.array_equal(got["kept_idx"], want["kept_idx"]) and np.array_equal(got["scores"], want["scores"])
    st.keep(got["kept_idx"])
    assert st.n_keys == 50
    assert np.array_equal(st.k, want["k_out"]) and np.array_equal(st.v, want["v_out"])
    assert np.array_equal(st.v_scale, want["v_scale_out"]) and np.array_equal(st.k_scale, ks)


def test_quantised_stream_with_unit_scales_walks_with_the_bf16_stream(oracle):
    """E4M3 values are bf16 values: with all scales one, three events of the quantised driver keep the same rows
    as the bf16 driver on the decoded values, and the caches stay decodings of one another."""
    from oracle import ea_quant
    from oracle.ea_stream import QuantStreamOracle, StreamOracle
    to_bf16 = lambda codes: (ea_quant.e4m3_decode(codes).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    q, kq, ks, vq, vs = _quant_case(22, U=1, n=160, W=12)
    ks[:], vs[:] = 1.0, 1.0
    qs = QuantStreamOracle(kq[:, :, :40], ks, vq[:, :, :40], vs[:, :, :40], window=12, budget=48)
    bs = StreamOracle(to_bf16(kq[:, :, :40]), to_bf16(vq[:, :, :40]), window=12, budget=48)
    rng = np.random.default_rng(5)
    for e in range(3):
        lo, hi = 40 + 40 * e, 80 + 40 * e
        qs.append(kq[:, :, lo:hi], vq[:, :, lo:hi], vs[:, :, lo:hi])
        bs.append(to_bf16(kq[:, :, lo:hi]), to_bf16(vq[:, :, lo:hi]))
        qn = (rng.normal(size=(1, 4, 7, 64)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
        qs.push_queries(qn)
        bs.push_queries(qn)
        a, b = qs.compress([hi], 8, 1e4, 0.02), bs.compress([hi], 8, 1e4, 0.02)
        np.testing.assert_allclose(a["scores"], b["scores"], rtol=1e-12, atol=0)
        assert np.array_equal(a["kept_idx"], b["kept_idx"])
        qs.keep(a["kept_idx"])
        bs.keep(b["kept_idx"])
        assert np.array_equal(to_bf16(qs.k), bs.k) and np.array_equal(to_bf16(qs.v), bs.v)
        assert (qs.v_scale == 1.0).all() and qs.v_scale.shape == (1, 2, qs.n_keys)


def test_quantised_adaptive_gather_against_the_c_routine_and_plain_indexing(oracle):
    """Codes are bytes: the ragged gather of code rows must equal the pinned C gather on the same bytes read as
    16-bit words, the scales must be the scales of the same tokens, and with the safeguard at the whole budget
    (every head keeps n_kept) the result is plain per-head indexing."""
    from oracle import ea_quant
    q, kq, ks, vq, vs = _quant_case(31, U=2, n=80)
    rng = np.random.default_rng(7)
    sc = rng.random((2, 2, 80)) * np.array([1.0, 4.0])[None, :, None]
    idx, off = oracle.select_adaptive(sc, 30, 6)
    assert (off[:, -1] == 60).all() and (np.diff(off, axis=1) != 30).any()          # genuinely ragged
    ko, vo, so = ea_quant.gather_adaptive(kq, vq, vs, idx, off)
    assert np.array_equal(ko.view(np.uint16), oracle.gather_adaptive(kq.view(np.uint16), idx, off))
    assert np.array_equal(vo.view(np.uint16), oracle.gather_adaptive(vq.view(np.uint16), idx, off))
    for u in range(2):
        for g in range(2):
            sl = slice(off[u, g], off[u, g + 1])
            assert np.array_equal(so[u, sl], vs[u, g][idx[u, sl]])
    idx_f, off_f = oracle.select_adaptive(sc, 30, 30)
    ko, vo, so = ea_quant.gather_adaptive(kq, vq, vs, idx_f, off_f)
    per_head = oracle.select(sc, 30).astype(np.int64)
    assert np.array_equal(ko.reshape(2, 2, 30, -1), np.take_along_axis(kq, per_head[..., None], axis=2))
    assert np.array_equal(so.reshape(2, 2, 30), np.take_along_axis(vs, per_head, axis=2))
