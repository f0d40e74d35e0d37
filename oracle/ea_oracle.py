"""ctypes front end of the fp64 CPU oracle (``ea_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It never touches the CUDA library and the CUDA
library never touches it.  Arrays are numpy; bf16 tensors travel as uint16 bit
patterns and are widened exactly inside the C code.

Parity status: pinned to the paper's definitions by the CPU test-suite; numeric
agreement with the authors' own code is unpinned (the paper prints no worked
example).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ea_oracle.c")
_LIB = os.path.join(_HERE, "libea_oracle.so")

ROPE_HALF_SPLIT, ROPE_INTERLEAVED = 0, 1
GROUP_MEAN_PROB, GROUP_SUM_PROB, GROUP_MEAN_LOGIT = 0, 1, 2
COV_POPULATION, COV_SAMPLE = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the library is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.eao_num_threads.restype = i32
        lib.eao_set_num_threads.argtypes = [i32]
        lib.eao_mean_cov.argtypes = [vp, i64, i32, i32, i32, vp, vp]
        lib.eao_rope_average.argtypes = [vp, i32, i32, f64, i32, vp, vp]
        lib.eao_apply_rope_average.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp]
        lib.eao_logits.argtypes = [vp, vp, vp, i32, i32, i32, i64, i32, vp]
        lib.eao_scores.argtypes = [vp, vp, i32, i32, i32, i64, i32, f64, i32, vp, vp]
        lib.eao_select.argtypes = [vp, i64, i64, i64, vp]
        lib.eao_gather.argtypes = [vp, vp, i64, i64, i64, i32, vp]
        lib.eao_n_kept.argtypes = [i64, f64]
        lib.eao_n_kept.restype = i64
        lib.eao_hidden_mean_cov.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp]
        lib.eao_hidden_mean_cov.restype = None
        lib.eao_scores_wo.argtypes = [vp, vp, vp, i32, i32, i32, i32, i64, i32, i32, f64, i32, vp]
        lib.eao_scores_wo.restype = None
        lib.eao_select_adaptive.argtypes = [vp, i64, i64, i64, i64, i64, vp, vp]
        lib.eao_gather_adaptive.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp]
        lib.eao_n_floor.argtypes = [i64, f64]
        lib.eao_n_floor.restype = i64
        for name in ("eao_set_num_threads", "eao_mean_cov", "eao_rope_average",
                     "eao_apply_rope_average", "eao_logits", "eao_scores", "eao_select",
                     "eao_gather", "eao_select_adaptive", "eao_gather_adaptive"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().eao_num_threads())


def set_num_threads(t: int) -> None:
    _load().eao_set_num_threads(int(t))


def n_kept(n: int, compression_ratio: float) -> int:
    return int(_load().eao_n_kept(int(n), float(compression_ratio)))


def mean_cov(q_win_bits, cov_norm=COV_POPULATION):
    """q_win_bits: uint16 [..., W, d] -> (mu [..., d], sigma [..., d, d]) float64."""
    q = _c(q_win_bits, np.uint16)
    *lead, W, d = q.shape
    nh = int(np.prod(lead)) if lead else 1
    mu = np.empty((nh, d), np.float64)
    sigma = np.empty((nh, d, d), np.float64)
    _load().eao_mean_cov(_p(q), nh, W, d, cov_norm, _p(mu), _p(sigma))
    return mu.reshape(*lead, d), sigma.reshape(*lead, d, d)


def rope_average(pos_next, n_future, rope_base, d):
    """pos_next: int64 [U] -> (cbar, sbar) float64 [U, d/2] (explicit sum over positions)."""
    pos = _c(pos_next, np.int64).reshape(-1)
    U = pos.shape[0]
    cbar = np.empty((U, d // 2), np.float64)
    sbar = np.empty((U, d // 2), np.float64)
    _load().eao_rope_average(_p(pos), U, int(n_future), float(rope_base), d, _p(cbar), _p(sbar))
    return cbar, sbar


def apply_rope_average(mu, sigma, cbar, sbar, layout=ROPE_HALF_SPLIT):
    """mu [U,Hq,d], sigma [U,Hq,d,d], cbar/sbar [U,d/2] -> (mu_bar, sigma_bar)."""
    mu = _c(mu, np.float64)
    sigma = _c(sigma, np.float64)
    cbar = _c(cbar, np.float64)
    sbar = _c(sbar, np.float64)
    U, Hq, d = mu.shape
    mu_bar = np.empty_like(mu)
    sigma_bar = np.empty_like(sigma)
    _load().eao_apply_rope_average(_p(mu), _p(sigma), _p(cbar), _p(sbar), U, Hq, d, layout,
                                   _p(mu_bar), _p(sigma_bar))
    return mu_bar, sigma_bar


def query_stats(q_win_bits, pos_next, n_future, rope_base, layout=ROPE_HALF_SPLIT,
                cov_norm=COV_POPULATION):
    """q_win_bits uint16 [U,Hq,W,d] -> (mu_bar [U,Hq,d], sigma_bar [U,Hq,d,d])."""
    d = q_win_bits.shape[-1]
    mu, sigma = mean_cov(q_win_bits, cov_norm)
    cbar, sbar = rope_average(pos_next, n_future, rope_base, d)
    return apply_rope_average(mu, sigma, cbar, sbar, layout)


def hidden_mean_cov(hidden_bits, w_q_bits, n_q_heads, cov_norm=COV_POPULATION):
    """hidden_bits uint16 [U, W, dm]; w_q_bits uint16 [sets, Hq*d, dm] (unit u uses set u // (U // sets))
    -> (mu [U,Hq,d], sigma [U,Hq,d,d]) of the pre-RoPE queries q = W_Q h."""
    H = _c(hidden_bits, np.uint16)
    Wq = _c(w_q_bits, np.uint16)
    U, W, dm = H.shape
    sets, rows, dm2 = Wq.shape
    assert dm2 == dm and rows % n_q_heads == 0
    d = rows // n_q_heads
    mu = np.empty((U, n_q_heads, d), np.float64)
    sigma = np.empty((U, n_q_heads, d, d), np.float64)
    _load().eao_hidden_mean_cov(_p(H), _p(Wq), U, sets, n_q_heads, W, d, dm, cov_norm, _p(mu), _p(sigma))
    return mu, sigma


def query_stats_hidden(hidden_bits, w_q_bits, n_q_heads, pos_next, n_future, rope_base,
                       layout=ROPE_HALF_SPLIT, cov_norm=COV_POPULATION):
    """Hidden states and query projections -> (mu_bar, sigma_bar) as query_stats gives them."""
    mu, sigma = hidden_mean_cov(hidden_bits, w_q_bits, n_q_heads, cov_norm)
    cbar, sbar = rope_average(pos_next, n_future, rope_base, mu.shape[-1])
    return apply_rope_average(mu, sigma, cbar, sbar, layout)


def logits(k_bits, mu_bar, sigma_bar):
    """k_bits uint16 [U,Hkv,n,d]; mu_bar [U,Hq,d]; sigma_bar [U,Hq,d,d] -> s [U,Hq,n]."""
    k = _c(k_bits, np.uint16)
    mu_bar = _c(mu_bar, np.float64)
    sigma_bar = _c(sigma_bar, np.float64)
    U, Hkv, n, d = k.shape
    Hq = mu_bar.shape[1]
    s = np.empty((U, Hq, n), np.float64)
    _load().eao_logits(_p(k), _p(mu_bar), _p(sigma_bar), U, Hq, Hkv, n, d, _p(s))
    return s


def scores(s, v_bits, eps, group_mode=GROUP_MEAN_PROB, return_attention=False):
    """s [U,Hq,n]; v_bits uint16 [U,Hkv,n,d] -> score [U,Hkv,n] (and a [U,Hkv,n])."""
    s = _c(s, np.float64)
    v = _c(v_bits, np.uint16)
    U, Hkv, n, d = v.shape
    Hq = s.shape[1]
    score = np.empty((U, Hkv, n), np.float64)
    a = np.empty((U, Hkv, n), np.float64) if return_attention else None
    _load().eao_scores(_p(s), _p(v), U, Hq, Hkv, n, d, float(eps), group_mode, _p(score),
                       _p(a) if a is not None else None)
    return (score, a) if return_attention else score


def scores_wo(s, v_bits, w_o_bits, eps, group_mode=GROUP_MEAN_PROB):
    """s [U,Hq,n]; v_bits uint16 [U,Hkv,n,d]; w_o_bits uint16 [sets, dm, Hq*d] -> score [U,Hkv,n]
    with ||W_o^h v|| in place of ||v|| (Eq. 9 as written); MEAN_PROB or SUM_PROB."""
    if group_mode == GROUP_MEAN_LOGIT:
        raise ValueError("the output-projection weighting is defined per query head")
    s = _c(s, np.float64)
    v = _c(v_bits, np.uint16)
    wo = _c(w_o_bits, np.uint16)
    U, Hkv, n, d = v.shape
    Hq = s.shape[1]
    sets, dm, cols = wo.shape
    assert cols == Hq * d
    score = np.empty((U, Hkv, n), np.float64)
    _load().eao_scores_wo(_p(s), _p(v), _p(wo), U, sets, Hq, Hkv, n, d, dm, float(eps), group_mode, _p(score))
    return score


def select(score, n_kept_):
    """score [..., n] -> kept indices int32 [..., n_kept], ascending."""
    sc = _c(score, np.float64)
    *lead, n = sc.shape
    nh = int(np.prod(lead)) if lead else 1
    idx = np.empty((nh, int(n_kept_)), np.int32)
    _load().eao_select(_p(sc), nh, n, int(n_kept_), _p(idx))
    return idx.reshape(*lead, int(n_kept_))


def gather(rows_bits, idx):
    """rows_bits uint16 [..., n, d]; idx int32 [..., n_kept] -> uint16 [..., n_kept, d]."""
    rows = _c(rows_bits, np.uint16)
    idx = _c(idx, np.int32)
    *lead, n, d = rows.shape
    nk = idx.shape[-1]
    nh = int(np.prod(lead)) if lead else 1
    out = np.empty((nh, nk, d), np.uint16)
    _load().eao_gather(_p(rows), _p(idx), nh, n, nk, d, _p(out))
    return out.reshape(*lead, nk, d)


def n_floor(n_kept_: int, alpha: float) -> int:
    return int(_load().eao_n_floor(int(n_kept_), float(alpha)))


def select_adaptive(score, n_kept_, n_floor_):
    """score [U, Hkv, n] -> (idx int32 [U, Hkv * n_kept], offsets int32 [U, Hkv + 1]).

    Head-adaptive eviction: each head keeps its n_floor best keys, the rest of the unit's budget of
    Hkv * n_kept goes to the best remaining pairs of the unit.
    """
    sc = _c(score, np.float64)
    U, Hkv, n = sc.shape
    if not 0 <= int(n_floor_) <= int(n_kept_) <= n:
        raise ValueError("need 0 <= n_floor <= n_kept <= n")
    idx = np.empty((U, Hkv * int(n_kept_)), np.int32)
    off = np.empty((U, Hkv + 1), np.int32)
    _load().eao_select_adaptive(_p(sc), U, Hkv, n, int(n_kept_), int(n_floor_), _p(idx), _p(off))
    return idx, off


def gather_adaptive(rows_bits, idx, offsets):
    """rows_bits uint16 [U, Hkv, n, d]; idx [U, B]; offsets [U, Hkv + 1] -> uint16 [U, B, d]."""
    rows = _c(rows_bits, np.uint16)
    idx = _c(idx, np.int32)
    off = _c(offsets, np.int32)
    U, Hkv, n, d = rows.shape
    B = idx.shape[1]
    out = np.empty((U, B, d), np.uint16)
    _load().eao_gather_adaptive(_p(rows), _p(idx), _p(off), U, Hkv, n, B, d, _p(out))
    return out


def compress(q_win_bits, k_bits, v_bits, pos_next, n_future, rope_base, eps, n_kept_,
             layout=ROPE_HALF_SPLIT, group_mode=GROUP_MEAN_PROB, cov_norm=COV_POPULATION):
    """Whole path; returns a dict of every intermediate."""
    mu_bar, sigma_bar = query_stats(q_win_bits, pos_next, n_future, rope_base, layout, cov_norm)
    s = logits(k_bits, mu_bar, sigma_bar)
    score = scores(s, v_bits, eps, group_mode)
    idx = select(score, n_kept_)
    return dict(mu_bar=mu_bar, sigma_bar=sigma_bar, logits=s, scores=score, kept_idx=idx,
                k_out=gather(k_bits, idx), v_out=gather(v_bits, idx))
