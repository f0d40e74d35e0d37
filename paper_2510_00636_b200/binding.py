"""Thin ctypes binding of ``libea.so`` (see ``include/ea.h``).

Argument marshalling only: torch supplies device memory and the current CUDA
stream; every step of the path runs in the library's kernels.  There is no
fallback: if the library is missing or the device is not a B200-class GPU the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libea.so")

ROPE_HALF_SPLIT, ROPE_INTERLEAVED = 0, 1
GROUP_MEAN_PROB, GROUP_SUM_PROB, GROUP_MEAN_LOGIT = 0, 1, 2
COV_POPULATION, COV_SAMPLE = 0, 1

EXPORTS = (
    "ea_version", "ea_status_string", "ea_workspace_bytes", "ea_n_kept", "ea_create", "ea_destroy",
    "ea_query_stats", "ea_score", "ea_select_compact", "ea_sync_status", "ea_profile_begin",
    "ea_profile_end", "ea_host_workspace_bytes", "ea_compress_host", "ea_query_stats_static",
    "ea_select_compact_adaptive", "ea_n_floor", "ea_query_stats_hidden", "ea_wo_gram", "ea_score_wo",
    "ea_select_compact_inplace", "ea_selftest_wait_timeout", "ea_last_cuda_error", "ea_set_sm_budget", "ea_set_side_sms", "ea_set_fused_stats", "ea_cache_append", "ea_window_push", "ea_query_stats_ring", "ea_score_q8", "ea_score_q8_scratch_bytes", "ea_select_compact_q8", "ea_cache_append_q8", "ea_select_compact_inplace_q8", "ea_select_compact_adaptive_q8", "ea_value_norms", "ea_score_vnorm", "ea_carry_f32_inplace", "ea_select_compact_inplace_unordered",
)
STATIC_MAX_ROPE_PAIRS = 16384


class EAError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = lib().ea_status_string(status).decode()
        detail = lib().ea_last_cuda_error().decode() if status == 4 else ""
        super().__init__(f"{where} failed: {name} ({status})" + (f": {detail}" if detail else ""))


class Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_units", "n_q_heads", "n_kv_heads", "head_dim", "n_keys", "window", "rope_layout",
        "group_mode", "cov_norm", "kv_capacity")]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2510_00636_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32, f64 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                                  ctypes.c_double)
        sp = ctypes.POINTER(Shape)
        L.ea_version.restype = ctypes.c_char_p
        L.ea_last_cuda_error.restype = ctypes.c_char_p
        L.ea_status_string.restype = ctypes.c_char_p
        L.ea_status_string.argtypes = [ctypes.c_int]
        L.ea_workspace_bytes.argtypes = [sp, ctypes.POINTER(ctypes.c_size_t)]
        L.ea_n_kept.argtypes = [i64, f64]
        L.ea_n_kept.restype = i64
        L.ea_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, ctypes.c_size_t]
        L.ea_destroy.argtypes = [vp]
        L.ea_query_stats.argtypes = [vp, sp, vp, vp, i32, f64, vp, vp, vp]
        L.ea_query_stats_static.argtypes = [sp, vp, vp, i32, f64, vp, vp, vp]
        L.ea_query_stats_static.restype = ctypes.c_int
        L.ea_query_stats_hidden.argtypes = [vp, sp, vp, vp, i32, i32, vp, vp, i32, f64, vp, vp, vp]
        L.ea_query_stats_hidden.restype = ctypes.c_int
        L.ea_score.argtypes = [vp, sp, vp, vp, vp, vp, f32, vp, vp, vp]
        L.ea_wo_gram.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp]
        L.ea_wo_gram.restype = ctypes.c_int
        L.ea_score_wo.argtypes = [vp, sp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp]
        L.ea_score_wo.restype = ctypes.c_int
        L.ea_select_compact.argtypes = [vp, sp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.ea_select_compact_adaptive.argtypes = [vp, sp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.ea_n_floor.argtypes = [i64, f64]
        L.ea_n_floor.restype = i64
        L.ea_select_compact_inplace.argtypes = [vp, sp, vp, i32, vp, vp, vp, vp]
        L.ea_select_compact_inplace.restype = ctypes.c_int
        L.ea_select_compact_inplace_unordered.argtypes = [vp, sp, vp, i32, vp, vp, vp, vp]
        L.ea_select_compact_inplace_unordered.restype = ctypes.c_int
        L.ea_selftest_wait_timeout.argtypes = [vp, i32, vp]
        L.ea_selftest_wait_timeout.restype = ctypes.c_int
        L.ea_cache_append.argtypes = [vp, sp, vp, vp, vp, vp, i32, vp]
        L.ea_window_push.argtypes = [vp, sp, vp, vp, vp, i32, vp]
        L.ea_query_stats_ring.argtypes = [vp, sp, vp, vp, vp, i32, f64, vp, vp, vp]
        for name in ("ea_cache_append", "ea_window_push", "ea_query_stats_ring"):
            getattr(L, name).restype = ctypes.c_int
        L.ea_score_q8.argtypes = [vp, sp, vp, vp, vp, vp, vp, vp, f32, vp, vp, vp, vp]
        L.ea_select_compact_q8.argtypes = [vp, sp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.ea_score_q8.restype = L.ea_select_compact_q8.restype = ctypes.c_int
        L.ea_score_q8_scratch_bytes.argtypes = [sp, ctypes.POINTER(ctypes.c_size_t)]
        L.ea_cache_append_q8.argtypes = [vp, sp, vp, vp, vp, vp, vp, vp, i32, vp]
        L.ea_select_compact_inplace_q8.argtypes = [vp, sp, vp, i32, vp, vp, vp, vp, i32, vp]
        L.ea_cache_append_q8.restype = L.ea_select_compact_inplace_q8.restype = ctypes.c_int
        L.ea_select_compact_adaptive_q8.argtypes = [vp, sp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.ea_select_compact_adaptive_q8.restype = ctypes.c_int
        L.ea_value_norms.argtypes = [vp, sp, vp, i32, i32, vp, vp]
        L.ea_score_vnorm.argtypes = [vp, sp, vp, vp, vp, vp, f32, vp, vp, vp]
        L.ea_carry_f32_inplace.argtypes = [vp, sp, vp, i32, vp, vp]
        L.ea_value_norms.restype = L.ea_score_vnorm.restype = L.ea_carry_f32_inplace.restype = ctypes.c_int
        L.ea_score_q8_scratch_bytes.restype = ctypes.c_int
        L.ea_set_fused_stats.argtypes = [vp, i32]
        L.ea_set_fused_stats.restype = ctypes.c_int
        L.ea_set_sm_budget.argtypes = [vp, i32]
        L.ea_set_side_sms.argtypes = [vp, i32]
        L.ea_set_side_sms.restype = ctypes.c_int
        L.ea_set_sm_budget.restype = ctypes.c_int
        L.ea_sync_status.argtypes = [vp, vp]
        L.ea_host_workspace_bytes.argtypes = [sp, i32, i32, ctypes.POINTER(ctypes.c_size_t)]
        L.ea_compress_host.argtypes = [vp, sp, vp, vp, vp, vp, i32, f64, f32, i32, i32, vp, vp, vp, vp, vp]
        L.ea_profile_begin.argtypes = [vp]
        L.ea_profile_end.argtypes = [vp, vp, ctypes.POINTER(f64), ctypes.POINTER(i64), ctypes.POINTER(i64)]
        for name in ("ea_workspace_bytes", "ea_create", "ea_destroy", "ea_query_stats", "ea_score",
                     "ea_select_compact", "ea_sync_status", "ea_profile_begin", "ea_profile_end",
                     "ea_host_workspace_bytes", "ea_compress_host", "ea_select_compact_adaptive"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise EAError(status, where)


def ea_n_kept(n_keys: int, compression_ratio: float) -> int:
    return int(lib().ea_n_kept(int(n_keys), float(compression_ratio)))


def ea_n_floor(n_kept: int, safeguard: float) -> int:
    return int(lib().ea_n_floor(int(n_kept), float(safeguard)))


def ea_workspace_bytes(shape: Shape) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ea_workspace_bytes(ctypes.byref(shape), ctypes.byref(out)), "ea_workspace_bytes")
    return int(out.value)


def make_shape(n_units, n_q_heads, n_kv_heads, head_dim, n_keys, window, rope_layout=ROPE_HALF_SPLIT,
               group_mode=GROUP_MEAN_PROB, cov_norm=COV_POPULATION, kv_capacity=0) -> Shape:
    return Shape(n_units, n_q_heads, n_kv_heads, head_dim, n_keys, window, rope_layout, group_mode,
                 cov_norm, kv_capacity)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _dev_tensor(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


class Context:
    """Owns an ``ea_ctx`` (its workspace lives on ``device``).

    Destroying a context frees device memory.  CUDA forbids that while a stream of the process is
    being captured into a graph (the capture is invalidated), so keep contexts alive across a
    capture and run ``gc.collect()`` before opening one if unreferenced contexts may be waiting
    for the garbage collector."""

    def __init__(self, device: int | torch.device = 0, workspace_bytes: int = 0):
        self.device = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
        handle = ctypes.c_void_p()
        _check(lib().ea_create(ctypes.byref(handle), self.device.index or 0, int(workspace_bytes)),
               "ea_create")
        self._h = handle
        self.workspace_bytes = int(workspace_bytes)

    @classmethod
    def for_shape(cls, shape: Shape, device=0) -> "Context":
        return cls(device, ea_workspace_bytes(shape))

    def close(self):
        if getattr(self, "_h", None):
            lib().ea_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sync_status(self):
        _check(lib().ea_sync_status(self._h, _stream(self.device)), "ea_sync_status")

    def selftest_wait_timeout(self, limit_us: int = 200):
        """Launch the self-test kernel whose bounded wait runs out (see ``ea_selftest_wait_timeout``)."""
        _check(lib().ea_selftest_wait_timeout(self._h, int(limit_us), _stream(self.device)),
               "ea_selftest_wait_timeout")

    def set_sm_budget(self, n_sms: int = 0):
        """Limit the persistent log-score kernel to ``n_sms`` SMs (0: all of them)."""
        _check(lib().ea_set_sm_budget(self._h, int(n_sms)), "ea_set_sm_budget")

    def set_side_sms(self, n_sms: int = 0):
        """Run the value-norm pass of ``ea_score`` on ``n_sms`` SMs beside the log-score kernel (0: off)."""
        _check(lib().ea_set_side_sms(self._h, int(n_sms)), "ea_set_side_sms")

    def set_fused_stats(self, on: bool = True):
        """Statistics calls also write the log-score kernel's operand; ``ea_score`` may then be called without
        ``mu_bar`` / ``sigma_bar`` (see ``ea_set_fused_stats``)."""
        _check(lib().ea_set_fused_stats(self._h, int(bool(on))), "ea_set_fused_stats")

    def profile_begin(self):
        _check(lib().ea_profile_begin(self._h), "ea_profile_begin")

    def profile_end(self):
        """-> (device ms summed over the timed log-score launches, their count, all kernel launches)."""
        ms, timed, total = ctypes.c_double(0), ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib().ea_profile_end(self._h, _stream(self.device), ctypes.byref(ms), ctypes.byref(timed),
                                    ctypes.byref(total)), "ea_profile_end")
        return ms.value, timed.value, total.value


def ea_query_stats(ctx: Context, shape: Shape, q_win, pos_next, n_future: int, rope_base: float,
                   mu_bar=None, sigma_bar=None, want_sigma: bool = True):
    """q_win bf16 [U,Hq,W,d], pos_next int64 [U] (device) -> (mu_bar [U,Hq,d], sigma_bar [U,Hq,d,d]).
    ``want_sigma=False`` (fused statistics only) leaves sigma_bar out: returns (mu_bar, None)."""
    _dev_tensor(q_win, torch.bfloat16, "q_win")
    _dev_tensor(pos_next, torch.int64, "pos_next")
    U, Hq, d = shape.n_units, shape.n_q_heads, shape.head_dim
    if mu_bar is None:
        mu_bar = torch.empty((U, Hq, d), dtype=torch.float32, device=q_win.device)
    if sigma_bar is None and want_sigma:
        sigma_bar = torch.empty((U, Hq, d, d), dtype=torch.float32, device=q_win.device)
    _check(lib().ea_query_stats(ctx._h, ctypes.byref(shape), _ptr(q_win), _ptr(pos_next), int(n_future),
                                float(rope_base), _ptr(mu_bar), _ptr(sigma_bar), _stream(ctx.device)),
           "ea_query_stats")
    return mu_bar, sigma_bar


def ea_cache_append(ctx: Context, shape: Shape, k, v, k_new, v_new):
    """Append ``k_new, v_new`` [U,Hkv,n_new,d] behind the ``shape.n_keys`` rows each head holds in ``k, v``
    [U,Hkv,kv_capacity,d] (in place)."""
    for t, name in ((k, "k"), (v, "v"), (k_new, "k_new"), (v_new, "v_new")):
        _dev_tensor(t, torch.bfloat16, name)
    _check(lib().ea_cache_append(ctx._h, ctypes.byref(shape), _ptr(k), _ptr(v), _ptr(k_new), _ptr(v_new),
                                 int(k_new.shape[2]), _stream(ctx.device)), "ea_cache_append")


def ea_cache_append_q8(ctx: Context, shape: Shape, k_q8, v_q8, v_scale, k_new, v_new, v_scale_new):
    """Append code rows ``k_new, v_new`` uint8 [U,Hkv,n_new,d] and their value scales [U,Hkv,n_new] behind the
    ``shape.n_keys`` rows each head holds in ``k_q8, v_q8`` [U,Hkv,kv_capacity,d] and ``v_scale`` (in place)."""
    for t, name in ((k_q8, "k_q8"), (v_q8, "v_q8"), (k_new, "k_new"), (v_new, "v_new")):
        _dev_tensor(t, torch.uint8, name)
    _dev_tensor(v_scale, torch.float32, "v_scale")
    _dev_tensor(v_scale_new, torch.float32, "v_scale_new")
    _check(lib().ea_cache_append_q8(ctx._h, ctypes.byref(shape), _ptr(k_q8), _ptr(v_q8), _ptr(v_scale), _ptr(k_new),
                                    _ptr(v_new), _ptr(v_scale_new), int(k_new.shape[2]), _stream(ctx.device)),
           "ea_cache_append_q8")


def ea_window_push(ctx: Context, shape: Shape, q_ring, ring_pushed, q_new):
    """Push ``q_new`` [U,Hq,n_new,d] into the ring ``q_ring`` [U,Hq,W,d]; ``ring_pushed`` int64 [U] (device) counts."""
    _dev_tensor(q_ring, torch.bfloat16, "q_ring")
    _dev_tensor(q_new, torch.bfloat16, "q_new")
    _dev_tensor(ring_pushed, torch.int64, "ring_pushed")
    _check(lib().ea_window_push(ctx._h, ctypes.byref(shape), _ptr(q_ring), _ptr(ring_pushed), _ptr(q_new),
                                int(q_new.shape[2]), _stream(ctx.device)), "ea_window_push")


def ea_query_stats_ring(ctx: Context, shape: Shape, q_ring, ring_pushed, pos_next, n_future: int, rope_base: float,
                        mu_bar=None, sigma_bar=None, want_sigma: bool = True):
    """``ea_query_stats`` over the rows a window ring holds -> (mu_bar, sigma_bar)."""
    _dev_tensor(q_ring, torch.bfloat16, "q_ring")
    _dev_tensor(ring_pushed, torch.int64, "ring_pushed")
    _dev_tensor(pos_next, torch.int64, "pos_next")
    U, Hq, d = shape.n_units, shape.n_q_heads, shape.head_dim
    if mu_bar is None:
        mu_bar = torch.empty((U, Hq, d), dtype=torch.float32, device=q_ring.device)
    if sigma_bar is None and want_sigma:
        sigma_bar = torch.empty((U, Hq, d, d), dtype=torch.float32, device=q_ring.device)
    _check(lib().ea_query_stats_ring(ctx._h, ctypes.byref(shape), _ptr(q_ring), _ptr(ring_pushed), _ptr(pos_next),
                                     int(n_future), float(rope_base), _ptr(mu_bar), _ptr(sigma_bar),
                                     _stream(ctx.device)), "ea_query_stats_ring")
    return mu_bar, sigma_bar


def ea_query_stats_hidden(ctx: Context, shape: Shape, hidden, w_q, pos_next, n_future: int, rope_base: float,
                          q_scratch=None, mu_bar=None, sigma_bar=None):
    """hidden bf16 [U,W,d_model], w_q bf16 [sets, Hq*d, d_model] -> (mu_bar, sigma_bar, q_scratch fp32 [U,Hq,W,d])."""
    _dev_tensor(hidden, torch.bfloat16, "hidden")
    _dev_tensor(w_q, torch.bfloat16, "w_q")
    _dev_tensor(pos_next, torch.int64, "pos_next")
    U, Hq, d, W = shape.n_units, shape.n_q_heads, shape.head_dim, shape.window
    d_model, n_sets = hidden.shape[-1], w_q.shape[0]
    dev = hidden.device
    if q_scratch is None:
        q_scratch = torch.empty((U, Hq, W, d), dtype=torch.float32, device=dev)
    if mu_bar is None:
        mu_bar = torch.empty((U, Hq, d), dtype=torch.float32, device=dev)
    if sigma_bar is None:
        sigma_bar = torch.empty((U, Hq, d, d), dtype=torch.float32, device=dev)
    _check(lib().ea_query_stats_hidden(ctx._h, ctypes.byref(shape), _ptr(hidden), _ptr(w_q), int(d_model),
                                       int(n_sets), _ptr(q_scratch), _ptr(pos_next), int(n_future),
                                       float(rope_base), _ptr(mu_bar), _ptr(sigma_bar), _stream(ctx.device)),
           "ea_query_stats_hidden")
    return mu_bar, sigma_bar, q_scratch


def ea_query_stats_static(shape: Shape, q_win, pos_next, n_future: int, rope_base: float, mu_bar, sigma_bar):
    """``ea_query_stats`` without a context: for callers that must not allocate device memory.

    The library call itself allocates nothing, so the outputs are NOT created here: the caller
    hands in ``mu_bar`` [U,Hq,d] and ``sigma_bar`` [U,Hq,d,d] (fp32, on the device of ``q_win``).
    Works on the tensors' device, which must be the current one; at most
    ``STATIC_MAX_ROPE_PAIRS`` (unit, channel pair) combinations per call.
    """
    _dev_tensor(q_win, torch.bfloat16, "q_win")
    _dev_tensor(pos_next, torch.int64, "pos_next")
    _dev_tensor(mu_bar, torch.float32, "mu_bar")
    _dev_tensor(sigma_bar, torch.float32, "sigma_bar")
    with torch.cuda.device(q_win.device):
        _check(lib().ea_query_stats_static(ctypes.byref(shape), _ptr(q_win), _ptr(pos_next), int(n_future),
                                           float(rope_base), _ptr(mu_bar), _ptr(sigma_bar),
                                           _stream(q_win.device)), "ea_query_stats_static")
    return mu_bar, sigma_bar


def ea_score(ctx: Context, shape: Shape, k, v, mu_bar, sigma_bar, epsilon: float, scores=None,
             logits=None, want_logits: bool = False):
    """k, v bf16 [U,Hkv,n,d] -> scores fp32 [U,Hkv,n] (and the log-scores [U,Hq,n] if asked)."""
    _dev_tensor(k, torch.bfloat16, "k")
    _dev_tensor(v, torch.bfloat16, "v")
    if sigma_bar is not None:                       # (None, None): the operand of a fused statistics call
        _dev_tensor(mu_bar, torch.float32, "mu_bar")
        _dev_tensor(sigma_bar, torch.float32, "sigma_bar")
    U, Hq, Hkv, n = shape.n_units, shape.n_q_heads, shape.n_kv_heads, shape.n_keys
    if scores is None:
        scores = torch.empty((U, Hkv, n), dtype=torch.float32, device=k.device)
    if logits is None and want_logits:
        logits = torch.empty((U, Hq, n), dtype=torch.float32, device=k.device)
    _check(lib().ea_score(ctx._h, ctypes.byref(shape), _ptr(k), _ptr(v), _ptr(mu_bar), _ptr(sigma_bar),
                          float(epsilon), _ptr(scores), _ptr(logits), _stream(ctx.device)), "ea_score")
    return (scores, logits) if (want_logits or logits is not None) else scores


def ea_value_norms(ctx: Context, shape: Shape, v, first_row: int, n_rows: int, v_norm):
    """``v_norm[u,g,i] = ||v[u,g,i]||`` for ``first_row <= i < first_row + n_rows``; v bf16 [U,Hkv,cap,d], v_norm fp32
    [U,Hkv,cap] (written in place)."""
    _dev_tensor(v, torch.bfloat16, "v")
    _dev_tensor(v_norm, torch.float32, "v_norm")
    _check(lib().ea_value_norms(ctx._h, ctypes.byref(shape), _ptr(v), int(first_row), int(n_rows), _ptr(v_norm),
                                _stream(ctx.device)), "ea_value_norms")


def ea_score_vnorm(ctx: Context, shape: Shape, k, v_norm, mu_bar, sigma_bar, epsilon: float, scores=None, logits=None,
                   want_logits: bool = False):
    """``ea_score`` with the carried value norms ``v_norm`` fp32 [U,Hkv,cap] in place of the value rows."""
    _dev_tensor(k, torch.bfloat16, "k")
    _dev_tensor(v_norm, torch.float32, "v_norm")
    U, Hq, Hkv, n = shape.n_units, shape.n_q_heads, shape.n_kv_heads, shape.n_keys
    if scores is None:
        scores = torch.empty((U, Hkv, n), dtype=torch.float32, device=k.device)
    if logits is None and want_logits:
        logits = torch.empty((U, Hq, n), dtype=torch.float32, device=k.device)
    _check(lib().ea_score_vnorm(ctx._h, ctypes.byref(shape), _ptr(k), _ptr(v_norm), _ptr(mu_bar), _ptr(sigma_bar),
                                float(epsilon), _ptr(scores), _ptr(logits), _stream(ctx.device)), "ea_score_vnorm")
    return (scores, logits) if (want_logits or logits is not None) else scores


def ea_carry_f32_inplace(ctx: Context, shape: Shape, kept_idx, n_kept: int, values):
    """``values[u,g,j] <- values[u,g,kept_idx[u,g,j]]`` for ``j < n_kept`` (in place), with the ``kept_idx`` an in-place
    compaction returned."""
    _dev_tensor(kept_idx, torch.int32, "kept_idx")
    _dev_tensor(values, torch.float32, "values")
    _check(lib().ea_carry_f32_inplace(ctx._h, ctypes.byref(shape), _ptr(kept_idx), int(n_kept), _ptr(values),
                                      _stream(ctx.device)), "ea_carry_f32_inplace")


def score_q8_scratch_bytes(shape: Shape) -> int:
    """Bytes of k_scratch ea_score_q8 needs for this shape (0: none)."""
    out = ctypes.c_size_t(0)
    _check(lib().ea_score_q8_scratch_bytes(ctypes.byref(shape), ctypes.byref(out)), "ea_score_q8_scratch_bytes")
    return int(out.value)


def ea_score_q8(ctx: Context, shape: Shape, k_q8, k_scale, v_q8, v_scale, mu_bar, sigma_bar, epsilon: float,
                k_scratch=None, scores=None, logits=None, want_logits: bool = False):
    """Scores of a quantised cache: k_q8, v_q8 uint8 [U,Hkv,cap,d] (E4M3 codes), k_scale fp32 [U,Hkv,d],
    v_scale fp32 [U,Hkv,cap] (cap = kv_capacity, or n) -> scores fp32 [U,Hkv,n] (and the log-scores if asked)."""
    _dev_tensor(k_q8, torch.uint8, "k_q8")
    _dev_tensor(v_q8, torch.uint8, "v_q8")
    _dev_tensor(k_scale, torch.float32, "k_scale")
    _dev_tensor(v_scale, torch.float32, "v_scale")
    U, Hq, Hkv, n, d = shape.n_units, shape.n_q_heads, shape.n_kv_heads, shape.n_keys, shape.head_dim
    dev = k_q8.device
    if k_scratch is None and score_q8_scratch_bytes(shape) > 0:
        # only where the tensor-core kernel does not widen the codes itself
        k_scratch = torch.empty((U, Hkv, shape.kv_capacity or n, d), dtype=torch.bfloat16, device=dev)
    if scores is None:
        scores = torch.empty((U, Hkv, n), dtype=torch.float32, device=dev)
    if logits is None and want_logits:
        logits = torch.empty((U, Hq, n), dtype=torch.float32, device=dev)
    _check(lib().ea_score_q8(ctx._h, ctypes.byref(shape), _ptr(k_q8), _ptr(k_scale), _ptr(v_q8), _ptr(v_scale),
                             _ptr(mu_bar), _ptr(sigma_bar), float(epsilon), _ptr(k_scratch), _ptr(scores),
                             _ptr(logits), _stream(ctx.device)), "ea_score_q8")
    return (scores, logits) if (want_logits or logits is not None) else scores


def ea_select_compact_q8(ctx: Context, shape: Shape, scores, n_kept: int, k_q8, v_q8, v_scale, out=None):
    """-> (kept_idx int32 [U,Hkv,n_kept], k_out, v_out uint8 [U,Hkv,n_kept,d], v_scale_out fp32 [U,Hkv,n_kept]);
    ``out`` may hand in these four tensors."""
    _dev_tensor(scores, torch.float32, "scores")
    U, Hkv, d = shape.n_units, shape.n_kv_heads, shape.head_dim
    dev = scores.device
    if out is not None:
        idx, k_out, v_out, vs_out = out
    else:
        idx = torch.empty((U, Hkv, n_kept), dtype=torch.int32, device=dev)
        k_out = torch.empty((U, Hkv, n_kept, d), dtype=torch.uint8, device=dev)
        v_out = torch.empty_like(k_out)
        vs_out = torch.empty((U, Hkv, n_kept), dtype=torch.float32, device=dev)
    _check(lib().ea_select_compact_q8(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), _ptr(k_q8), _ptr(v_q8),
                                      _ptr(v_scale), _ptr(idx), _ptr(k_out), _ptr(v_out), _ptr(vs_out),
                                      _stream(ctx.device)), "ea_select_compact_q8")
    return idx, k_out, v_out, vs_out


def ea_wo_gram(ctx: Context, w_o, n_q_heads: int, head_dim: int, wo_gram=None):
    """w_o bf16 [sets, d_model, Hq*d] -> Gram matrices fp32 [sets, Hq, d, d] of the per-head slices."""
    _dev_tensor(w_o, torch.bfloat16, "w_o")
    sets, d_model, cols = w_o.shape
    if cols != n_q_heads * head_dim:
        raise ValueError("w_o must be [sets, d_model, Hq * d]")
    if wo_gram is None:
        wo_gram = torch.empty((sets, n_q_heads, head_dim, head_dim), dtype=torch.float32, device=w_o.device)
    _check(lib().ea_wo_gram(ctx._h, _ptr(w_o), int(d_model), int(sets), int(n_q_heads), int(head_dim),
                            _ptr(wo_gram), _stream(ctx.device)), "ea_wo_gram")
    return wo_gram


def ea_score_wo(ctx: Context, shape: Shape, k, v, mu_bar, sigma_bar, wo_gram, epsilon: float, scores=None,
                wo_scratch=None, logits=None, want_logits: bool = False):
    """As ea_score with ||W_o^h v|| per query head in place of ||v||; returns (scores, wo_scratch[, logits])."""
    _dev_tensor(k, torch.bfloat16, "k")
    _dev_tensor(v, torch.bfloat16, "v")
    _dev_tensor(mu_bar, torch.float32, "mu_bar")
    _dev_tensor(sigma_bar, torch.float32, "sigma_bar")
    _dev_tensor(wo_gram, torch.float32, "wo_gram")
    U, Hq, Hkv, n = shape.n_units, shape.n_q_heads, shape.n_kv_heads, shape.n_keys
    if scores is None:
        scores = torch.empty((U, Hkv, n), dtype=torch.float32, device=k.device)
    if wo_scratch is None:
        wo_scratch = torch.empty((U, Hq, n), dtype=torch.float32, device=k.device)
    if logits is None and want_logits:
        logits = torch.empty((U, Hq, n), dtype=torch.float32, device=k.device)
    _check(lib().ea_score_wo(ctx._h, ctypes.byref(shape), _ptr(k), _ptr(v), _ptr(mu_bar), _ptr(sigma_bar),
                             _ptr(wo_gram), int(wo_gram.shape[0]), float(epsilon), _ptr(wo_scratch), _ptr(scores),
                             _ptr(logits), _stream(ctx.device)), "ea_score_wo")
    return (scores, wo_scratch, logits) if want_logits else (scores, wo_scratch)


def ea_select_compact(ctx: Context, shape: Shape, scores, n_kept: int, k=None, v=None, kept_idx=None,
                      k_out=None, v_out=None, gather: bool = True):
    """scores fp32 [U,Hkv,n] -> (kept_idx int32 [U,Hkv,n_kept], k_out, v_out bf16 [U,Hkv,n_kept,d])."""
    _dev_tensor(scores, torch.float32, "scores")
    U, Hkv, d = shape.n_units, shape.n_kv_heads, shape.head_dim
    if kept_idx is None:
        kept_idx = torch.empty((U, Hkv, max(n_kept, 0)), dtype=torch.int32, device=scores.device)
    if gather:
        _dev_tensor(k, torch.bfloat16, "k")
        _dev_tensor(v, torch.bfloat16, "v")
        if k_out is None:
            k_out = torch.empty((U, Hkv, max(n_kept, 0), d), dtype=torch.bfloat16, device=scores.device)
        if v_out is None:
            v_out = torch.empty((U, Hkv, max(n_kept, 0), d), dtype=torch.bfloat16, device=scores.device)
    _check(lib().ea_select_compact(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), _ptr(k),
                                   _ptr(v), _ptr(kept_idx), _ptr(k_out), _ptr(v_out),
                                   _stream(ctx.device)), "ea_select_compact")
    return kept_idx, k_out, v_out


def ea_select_compact_inplace_unordered(ctx: Context, shape: Shape, scores, n_kept: int, k, v, kept_idx=None):
    """Selection, then only the kept rows beyond ``n_kept`` move, into the evicted positions below it (in place).
    Returns the position, before the call, of the row at each of the first ``n_kept`` positions afterwards."""
    _dev_tensor(scores, torch.float32, "scores")
    _dev_tensor(k, torch.bfloat16, "k")
    _dev_tensor(v, torch.bfloat16, "v")
    if kept_idx is None:
        kept_idx = torch.empty((shape.n_units, shape.n_kv_heads, max(n_kept, 0)), dtype=torch.int32,
                               device=scores.device)
    _check(lib().ea_select_compact_inplace_unordered(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), _ptr(k),
                                                     _ptr(v), _ptr(kept_idx), _stream(ctx.device)),
           "ea_select_compact_inplace_unordered")
    return kept_idx


def ea_select_compact_inplace_q8(ctx: Context, shape: Shape, scores, n_kept: int, k_q8, v_q8, v_scale, kept_idx=None,
                                 unordered: bool = False):
    """In-place compaction of a quantised cache (code rows and the value scales of their tokens); ordered as
    ``ea_select_compact_inplace`` or, with ``unordered``, as ``ea_select_compact_inplace_unordered``."""
    _dev_tensor(scores, torch.float32, "scores")
    _dev_tensor(k_q8, torch.uint8, "k_q8")
    _dev_tensor(v_q8, torch.uint8, "v_q8")
    _dev_tensor(v_scale, torch.float32, "v_scale")
    if kept_idx is None:
        kept_idx = torch.empty((shape.n_units, shape.n_kv_heads, max(n_kept, 0)), dtype=torch.int32,
                               device=scores.device)
    _check(lib().ea_select_compact_inplace_q8(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), _ptr(k_q8),
                                              _ptr(v_q8), _ptr(v_scale), _ptr(kept_idx), int(bool(unordered)),
                                              _stream(ctx.device)), "ea_select_compact_inplace_q8")
    return kept_idx


def ea_select_compact_inplace(ctx: Context, shape: Shape, scores, n_kept: int, k, v, kept_idx=None):
    """Selection, then the kept rows of every head move to the front of k and v (modified in place)."""
    _dev_tensor(scores, torch.float32, "scores")
    _dev_tensor(k, torch.bfloat16, "k")
    _dev_tensor(v, torch.bfloat16, "v")
    if kept_idx is None:
        kept_idx = torch.empty((shape.n_units, shape.n_kv_heads, max(n_kept, 0)), dtype=torch.int32,
                               device=scores.device)
    _check(lib().ea_select_compact_inplace(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), _ptr(k), _ptr(v),
                                           _ptr(kept_idx), _stream(ctx.device)), "ea_select_compact_inplace")
    return kept_idx


def ea_select_compact_adaptive(ctx: Context, shape: Shape, scores, n_kept: int, n_floor: int, k=None, v=None,
                               kept_idx=None, head_offsets=None, k_out=None, v_out=None, gather: bool = True):
    """scores fp32 [U,Hkv,n] -> (kept_idx int32 [U,Hkv*n_kept], head_offsets int32 [U,Hkv+1],
    k_out, v_out bf16 [U,Hkv*n_kept,d]); head g of unit u owns kept_idx[u, off[u,g]:off[u,g+1]]."""
    _dev_tensor(scores, torch.float32, "scores")
    U, Hkv, d = shape.n_units, shape.n_kv_heads, shape.head_dim
    B = Hkv * max(n_kept, 0)
    if kept_idx is None:
        kept_idx = torch.empty((U, B), dtype=torch.int32, device=scores.device)
    if head_offsets is None:
        head_offsets = torch.empty((U, Hkv + 1), dtype=torch.int32, device=scores.device)
    if gather:
        _dev_tensor(k, torch.bfloat16, "k")
        _dev_tensor(v, torch.bfloat16, "v")
        if k_out is None:
            k_out = torch.empty((U, B, d), dtype=torch.bfloat16, device=scores.device)
        if v_out is None:
            v_out = torch.empty((U, B, d), dtype=torch.bfloat16, device=scores.device)
    _check(lib().ea_select_compact_adaptive(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), int(n_floor),
                                            _ptr(k), _ptr(v), _ptr(kept_idx), _ptr(head_offsets), _ptr(k_out),
                                            _ptr(v_out), _stream(ctx.device)), "ea_select_compact_adaptive")
    return kept_idx, head_offsets, k_out, v_out


def ea_select_compact_adaptive_q8(ctx: Context, shape: Shape, scores, n_kept: int, n_floor: int, k_q8, v_q8, v_scale):
    """Head-adaptive eviction on a quantised cache -> (kept_idx [U,Hkv*n_kept], head_offsets [U,Hkv+1],
    k_out, v_out uint8 [U,Hkv*n_kept,d], v_scale_out fp32 [U,Hkv*n_kept])."""
    _dev_tensor(scores, torch.float32, "scores")
    _dev_tensor(k_q8, torch.uint8, "k_q8")
    _dev_tensor(v_q8, torch.uint8, "v_q8")
    _dev_tensor(v_scale, torch.float32, "v_scale")
    U, Hkv, d = shape.n_units, shape.n_kv_heads, shape.head_dim
    B, dev = Hkv * max(n_kept, 0), scores.device
    kept_idx = torch.empty((U, B), dtype=torch.int32, device=dev)
    head_offsets = torch.empty((U, Hkv + 1), dtype=torch.int32, device=dev)
    k_out = torch.empty((U, B, d), dtype=torch.uint8, device=dev)
    v_out = torch.empty((U, B, d), dtype=torch.uint8, device=dev)
    v_scale_out = torch.empty((U, B), dtype=torch.float32, device=dev)
    _check(lib().ea_select_compact_adaptive_q8(ctx._h, ctypes.byref(shape), _ptr(scores), int(n_kept), int(n_floor),
                                               _ptr(k_q8), _ptr(v_q8), _ptr(v_scale), _ptr(kept_idx),
                                               _ptr(head_offsets), _ptr(k_out), _ptr(v_out), _ptr(v_scale_out),
                                               _stream(ctx.device)), "ea_select_compact_adaptive_q8")
    return kept_idx, head_offsets, k_out, v_out, v_scale_out


@dataclass
class Compressed:
    mu_bar: torch.Tensor
    sigma_bar: torch.Tensor
    scores: torch.Tensor
    logits: torch.Tensor | None
    kept_idx: torch.Tensor
    k_out: torch.Tensor
    v_out: torch.Tensor


def compress(ctx: Context, shape: Shape, q_win, k, v, pos_next, n_future, rope_base, epsilon, n_kept,
             want_logits: bool = False) -> Compressed:
    """The three calls back to back on the current stream."""
    mu_bar, sigma_bar = ea_query_stats(ctx, shape, q_win, pos_next, n_future, rope_base)
    res = ea_score(ctx, shape, k, v, mu_bar, sigma_bar, epsilon, want_logits=want_logits)
    scores, logits = res if want_logits else (res, None)
    kept_idx, k_out, v_out = ea_select_compact(ctx, shape, scores, n_kept, k, v)
    return Compressed(mu_bar, sigma_bar, scores, logits, kept_idx, k_out, v_out)


def ea_host_workspace_bytes(shape: Shape, n_kept: int, units_per_chunk: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().ea_host_workspace_bytes(ctypes.byref(shape), int(n_kept), int(units_per_chunk),
                                         ctypes.byref(out)), "ea_host_workspace_bytes")
    return int(out.value)


def _host_tensor(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CPU tensor of {dtype}")
    return t


def ea_compress_host(ctx: Context, shape: Shape, q_win, k, v, pos_next, n_future, rope_base, epsilon,
                     n_kept: int, units_per_chunk: int = 1, kept_idx=None, k_out=None, v_out=None,
                     scores=None):
    """Whole routine on HOST tensors (pin them for overlapped copies).  Asynchronous: call
    ``ctx.sync_status()`` before reading the returned host tensors."""
    _host_tensor(q_win, torch.bfloat16, "q_win")
    _host_tensor(k, torch.bfloat16, "k")
    _host_tensor(v, torch.bfloat16, "v")
    _host_tensor(pos_next, torch.int64, "pos_next")
    U, Hkv, d = shape.n_units, shape.n_kv_heads, shape.head_dim
    pin = k.is_pinned()
    if kept_idx is None:
        kept_idx = torch.empty((U, Hkv, n_kept), dtype=torch.int32, pin_memory=pin)
    if k_out is None:
        k_out = torch.empty((U, Hkv, n_kept, d), dtype=torch.bfloat16, pin_memory=pin)
    if v_out is None:
        v_out = torch.empty((U, Hkv, n_kept, d), dtype=torch.bfloat16, pin_memory=pin)
    _check(lib().ea_compress_host(ctx._h, ctypes.byref(shape), _ptr(q_win), _ptr(k), _ptr(v),
                                  _ptr(pos_next), int(n_future), float(rope_base), float(epsilon),
                                  int(n_kept), int(units_per_chunk), _ptr(kept_idx), _ptr(k_out),
                                  _ptr(v_out), _ptr(scores), _stream(ctx.device)), "ea_compress_host")
    return kept_idx, k_out, v_out
