"""Host-side checks that need no GPU: the library builds, loads, exports what the header
declares, and its host-only arithmetic agrees with the oracle's."""
import ctypes
import os
import re

import numpy as np
import pytest

import parity
from paper_2510_00636_b200 import build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ea():
    build.build()
    from paper_2510_00636_b200 import binding
    binding.lib()
    return binding


def test_library_exports_every_declared_symbol(ea):
    header = open(os.path.join(ROOT, "include", "ea.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ea_[a-z_0-9]+)\s*\(", header))
    assert declared >= {"ea_query_stats", "ea_score", "ea_select_compact", "ea_create", "ea_destroy"}
    L = ea.lib()
    for name in declared:
        assert hasattr(L, name), f"{name} declared in ea.h but not exported"
    assert set(ea.EXPORTS) <= declared
    assert L.ea_version().startswith(b"ea-b200")


def test_n_kept_matches_oracle(ea, oracle):
    rng = np.random.default_rng(0)
    for n, r in [(512, 0.5), (8192, 0.5), (32768, 0.75), (131072, 0.875), (10, 0.7), (10, 0.9), (0, 0.5),
                 (5, 0.0), (5, 1.0), (5, 1.5), (5, -0.5)]:
        assert ea.ea_n_kept(n, r) == oracle.n_kept(n, r), (n, r)
    for _ in range(500):
        n, r = int(rng.integers(0, 1 << 20)), float(rng.random())
        assert ea.ea_n_kept(n, r) == oracle.n_kept(n, r) == int(n * (1 - r))


def test_workspace_bytes_and_shape_validation(ea):
    small = ea.ea_workspace_bytes(ea.make_shape(1, 4, 2, 64, 512, 64))
    big = ea.ea_workspace_bytes(ea.make_shape(48, 16, 8, 256, 131072, 256))
    assert 0 < small < big
    assert big >= 48 * 16 * 131072 * 4          # room for the fp32 log-scores
    assert big < 2 << 30
    for bad, status in [(ea.make_shape(1, 4, 3, 64, 512, 64), 1), (ea.make_shape(1, 4, 2, 96, 512, 64), 2),
                        (ea.make_shape(-1, 4, 2, 64, 512, 64), 1), (ea.make_shape(1, 4, 2, 64, 512, 64, 7), 1),
                        (ea.make_shape(1, 4, 2, 64, 512, 64, 0, 3), 1)]:
        with pytest.raises(ea.EAError) as e:
            ea.ea_workspace_bytes(bad)
        assert e.value.status == status
    assert ea.lib().ea_workspace_bytes(None, None) == 1


def test_null_context_is_rejected_without_touching_cuda(ea):
    L = ea.lib()
    shape = ea.make_shape(1, 4, 2, 64, 512, 64)
    assert L.ea_query_stats(None, ctypes.byref(shape), None, None, 512, 1e4, None, None, None) == 1
    assert L.ea_score(None, ctypes.byref(shape), None, None, None, None, 0.02, None, None, None) == 1
    assert L.ea_select_compact(None, ctypes.byref(shape), None, 1, None, None, None, None, None, None) == 1
    assert L.ea_sync_status(None, None) == 1
    assert L.ea_destroy(None) == 0
    assert L.ea_status_string(6) == b"EA_ERR_DEVICE_TIMEOUT"


def test_create_fails_cleanly_without_a_gpu(ea):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    status = ea.lib().ea_create(ctypes.byref(h), 0, 1024)
    assert status in (4, 5) and not h.value        # EA_ERR_CUDA / EA_ERR_NOT_SM100: no CPU fallback
    with pytest.raises(ea.EAError):
        ea.Context(0, 1024)


def test_decode_schedule():
    ev = inputs.decode_schedule()
    assert len(ev) == 28 and ev[0] == (2560, 2560, 2560) and ev[3] == (4096, 4096, 4096)
    assert ev[4] == (4608, 4608, 4096) and ev[-1] == (16384, 4608, 4096)
    assert sum(n for _, n, _ in ev) * 8 * 28 * 4 == 111_017_984


# ---------------------------------------------------------------- the tolerance protocol itself
def test_parity_protocol_accepts_small_and_rejects_large_deviations(oracle):
    cfg = inputs.CONFIGS[0].tempered(2.0)
    q, k, v, pos = inputs.generate_layer(cfg)
    qb, kb, vb = inputs.bits(q), inputs.bits(k), inputs.bits(v)
    ref = oracle.compress(qb, kb, vb, pos.numpy(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept)
    delta = parity.logit_error_bound(kb, ref["mu_bar"], ref["sigma_bar"], 24)
    assert delta.max() < 1e-3
    lo, hi = parity.score_range(ref["logits"], delta, vb, cfg.eps)
    assert np.all(lo <= ref["scores"]) and np.all(ref["scores"] <= hi)
    rng = np.random.default_rng(0)
    ok = ref["scores"] * (1 + 5e-3 * rng.uniform(-1, 1, ref["scores"].shape))
    assert parity.check_scores(ok, lo, hi) == (0, 0)
    off = ref["scores"].copy()
    off[0, 1, 17] *= 1.03
    assert parity.check_scores(off, lo, hi)[0] == 1
    assert parity.check_logits(ref["logits"] + 0.5 * delta, ref["logits"], delta)[0] == 0
    assert parity.check_logits(ref["logits"] * 1.02, ref["logits"], delta)[0] > 0
    # kept set: the oracle's own selection passes; swapping a clear winner for a clear loser fails
    idx = ref["kept_idx"].copy()
    assert parity.check_kept(idx, lo, hi, cfg.n_kept)[:2] == (0, 0)
    order = np.argsort(-ref["scores"][0, 0])
    best, worst = order[0], order[-1]
    row = [i for i in idx[0, 0] if i != best] + [worst]
    idx[0, 0] = np.sort(np.array(row, dtype=np.int32))
    missing, present, _ = parity.check_kept(idx, lo, hi, cfg.n_kept)
    assert missing == 1 and present == 1
    # a one-hot softmax (literal config) is flagged as unstable rather than silently passed
    cfg = inputs.CONFIGS[0]
    q, k, v, pos = inputs.generate_layer(cfg)
    kb, vb = inputs.bits(k), inputs.bits(v)
    ref = oracle.compress(inputs.bits(q), kb, vb, pos.numpy(), cfg.n_future, cfg.rope_base, cfg.eps, cfg.n_kept)
    delta = parity.logit_error_bound(kb, ref["mu_bar"], ref["sigma_bar"], 8)
    lo, hi = parity.score_range(ref["logits"], delta, vb, cfg.eps)
    assert np.all(lo <= ref["scores"] * (1 + 1e-12)) and np.all(ref["scores"] <= hi * (1 + 1e-12))
