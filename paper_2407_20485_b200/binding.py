"""Thin ctypes binding over ``liba2sf.so`` (see ``include/a2sf.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch supplies device memory and streams.  There is no fallback: if the
library has not been built this module raises on import.
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path
from typing import Optional

import torch

# A2SF_LIBRARY=debug selects the bounds-checked build (liba2sf_debug.so, see build.py)
_LIB_PATH = Path(__file__).resolve().parent / (
    "liba2sf_debug.so" if os.environ.get("A2SF_LIBRARY", "") == "debug" else "liba2sf.so")

A2SF_F32, A2SF_BF16, A2SF_F16 = 0, 1, 2
_DTYPE_CODE = {torch.float32: A2SF_F32, torch.bfloat16: A2SF_BF16, torch.float16: A2SF_F16}

A2SF_OK = 0
A2SF_ERR_INVALID_ARG, A2SF_ERR_UNSUPPORTED, A2SF_ERR_CUDA = -1, -2, -3
A2SF_ERR_TIMEOUT, A2SF_ERR_WORKSPACE = -4, -5


class a2sf_params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("d", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("budget", ctypes.c_int32), ("recent", ctypes.c_int32),
                ("alpha", ctypes.c_float), ("scale", ctypes.c_float), ("flags", ctypes.c_int32),
                ("score_window", ctypes.c_int32)]


class A2SFError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def _load():
    if not _LIB_PATH.exists():
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2407_20485_b200.build` (add --debug "
            "for the bounds-checked library) "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i32, i64, f32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                             ctypes.c_size_t)
    pp = ctypes.POINTER(a2sf_params)
    pvp = ctypes.POINTER(vp)
    sigs = {
        "a2sf_prefill_workspace_bytes": (sz, [pp, i32]),
        "a2sf_prefill": (ctypes.c_int, [pp, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, vp, sz, vp]),
        "a2sf_prefill_per_head": (ctypes.c_int, [pp, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, vp, vp, sz, vp]),
        "a2sf_rescore_per_head": (ctypes.c_int, [pp, i32, vp, vp, i64, i64, i64, vp, vp, vp, vp, vp, sz, vp]),
        "a2sf_decode_step_per_head": (ctypes.c_int, [vp, vp, vp, vp, vp, vp, vp, vp]),
        "a2sf_rescore_workspace_bytes": (sz, [pp, i32]),
        "a2sf_rescore": (ctypes.c_int, [pp, i32, vp, vp, i64, i64, i64, vp, vp, vp, vp, sz, vp]),
        "a2sf_prefill_static_scratch_max_rows": (sz, []),
        "a2sf_prefill_static_scratch": (ctypes.c_int, [pp, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp, vp]),
        "a2sf_prefill_host_workspace_bytes": (sz, [pp, i32]),
        "a2sf_prefill_host": (ctypes.c_int, [pp, i32, vp, vp, vp, vp, vp, vp, vp, sz,
                                             pvp, pvp, pvp, pvp, vp]),
        "a2sf_cache_bytes": (sz, [pp]),
        "a2sf_cache_create": (ctypes.c_int, [pp, vp, sz, pvp]),
        "a2sf_cache_destroy": (ctypes.c_int, [vp]),
        "a2sf_cache_load": (ctypes.c_int, [vp, i32, vp, vp, i64, i64, i64, vp, vp, vp]),
        "a2sf_decode_step": (ctypes.c_int, [vp, f32, vp, vp, vp, vp, vp, vp]),
        "a2sf_decode_step_host": (ctypes.c_int, [vp, f32, vp, vp, vp, vp, vp, vp]),
        "a2sf_cache_reset": (ctypes.c_int, [vp, vp]),
        "a2sf_prefill_group_workspace_bytes": (sz, [pp, i32, i32]),
        "a2sf_prefill_group": (ctypes.c_int, [pp, i32, i32, vp, i64, i64, i64, vp, vp, i64, i64, i64,
                                              vp, vp, vp, vp, vp, sz, vp]),
        "a2sf_decode_step_group": (ctypes.c_int, [vp, i32, f32, vp, vp, vp, vp, vp, vp]),
        "a2sf_ideal_similarity_workspace_bytes": (sz, [pp, i32]),
        "a2sf_ideal_similarity": (ctypes.c_int, [vp, f32, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, sz, vp]),
        "a2sf_score_window_bound": (ctypes.c_double, [f32, i32, i32]),
        "a2sf_decode_multi": (ctypes.c_int, [vp, f32, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp]),
        "a2sf_prefill_streaming": (ctypes.c_int, [vp, f32, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp]),
        "a2sf_cache_export": (ctypes.c_int, [vp] * 8),
        "a2sf_cache_import": (ctypes.c_int, [vp] * 8),
        "a2sf_kernel_launch_count": (ctypes.c_int64, []),
        "a2sf_last_device_status": (ctypes.c_int, [vp]),
        "a2sf_debug_build": (ctypes.c_int, []),
        "a2sf_debug_violations": (ctypes.c_int, [ctypes.POINTER(ctypes.c_int64), vp]),
        "a2sf_select": (ctypes.c_int, [ctypes.POINTER(a2sf_params), ctypes.c_int32, vp, vp, vp]),
        "a2sf_selftest_bounded_wait": (ctypes.c_int, [ctypes.c_int32, ctypes.c_int64, vp, vp]),
        "a2sf_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib, tuple(sigs)


lib, EXPORTED = _load()


def status_string(status: int) -> str:
    return lib.a2sf_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != A2SF_OK:
        raise A2SFError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS = 1


def make_params(B: int, H: int, d: int, dtype: torch.dtype, budget: int, recent: int,
                alpha: float, scale: float = 0.0, flags: int = 0, score_window: int = 0) -> a2sf_params:
    return a2sf_params(B, H, d, _DTYPE_CODE[dtype], budget, recent, alpha, scale, flags, score_window)


def a2sf_score_window_bound(alpha: float, n: int, score_window: int) -> float:
    return float(lib.a2sf_score_window_bound(alpha, n, score_window))


def a2sf_kernel_launch_count() -> int:
    return int(lib.a2sf_kernel_launch_count())


def a2sf_last_device_status(stream=None) -> int:
    return int(lib.a2sf_last_device_status(_stream(stream)))


def a2sf_debug_build() -> bool:
    return bool(lib.a2sf_debug_build())


def a2sf_debug_violations(stream=None):
    """(count, kernel id, source line, index, bound) of the bounds-checked debug library since the
    last call; all zero in the release library."""
    rep = (ctypes.c_int64 * 4)()
    _check(lib.a2sf_debug_violations(rep, _stream(stream)), "a2sf_debug_violations")
    return int(rep[0]), int(rep[1]) >> 32, int(rep[1]) & 0xffffffff, int(rep[2]), int(rep[3])


def a2sf_select(p: a2sf_params, scores: torch.Tensor, kept_idx=None, stream=None) -> torch.Tensor:
    """Selection alone: the kept set of ``scores`` [B, H, n] (fp32, contiguous)."""
    assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.dim() == 3
    n = scores.shape[2]
    if kept_idx is None:
        kept_idx = torch.empty((p.B, p.H, min(n, p.budget)), dtype=torch.int32, device=scores.device)
    _check(lib.a2sf_select(ctypes.byref(p), n, _ptr(scores), _ptr(kept_idx), _stream(stream)), "a2sf_select")
    return kept_idx


def a2sf_selftest_bounded_wait(which: int, limit_cycles: int, stream=None) -> torch.Tensor:
    """Runs the bounded-wait self-test; returns the kernel's report (int64[4], on the device)."""
    report = torch.zeros((4,), dtype=torch.int64, device="cuda")
    _check(lib.a2sf_selftest_bounded_wait(which, limit_cycles, report.data_ptr(), _stream(stream)),
           "a2sf_selftest_bounded_wait")
    return report


def a2sf_prefill_workspace_bytes(p: a2sf_params, n: int) -> int:
    return int(lib.a2sf_prefill_workspace_bytes(ctypes.byref(p), n))


def a2sf_rescore_workspace_bytes(p: a2sf_params, n: int) -> int:
    return int(lib.a2sf_rescore_workspace_bytes(ctypes.byref(p), n))


def _strides(t: torch.Tensor):
    assert t.dim() == 4 and t.stride(3) == 1, "expected [B,H,n,d] with contiguous d"
    return t.stride(0), t.stride(1), t.stride(2)


def a2sf_prefill(p: a2sf_params, q, k, v, out=None, scores=None, kept_idx=None, lse=None,
                 workspace=None, stream=None, alphas=None):
    """q, k, v: device [B,H,n,d].  Returns (out, scores, kept_idx, lse).
    ``alphas``: optional device tensor [B,H] fp32 of per-head forgetting factors."""
    B, H, n, d = q.shape
    assert k.shape == q.shape and v.shape == q.shape
    assert _strides(k) == _strides(q) and _strides(v) == _strides(q)
    dev = q.device
    m = min(n, p.budget)
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=dev)
    assert _strides(out) == _strides(q)
    scores = torch.empty((B, H, n), dtype=torch.float32, device=dev) if scores is None else scores
    kept_idx = torch.empty((B, H, m), dtype=torch.int32, device=dev) if kept_idx is None else kept_idx
    lse = torch.empty((B, H, n), dtype=torch.float32, device=dev) if lse is None else lse
    if workspace is None:
        need = a2sf_prefill_workspace_bytes(p, n)
        workspace = torch.empty((max(need, 256),), dtype=torch.uint8, device=dev)
    sb, sh, st = _strides(q)
    if alphas is None:
        _check(lib.a2sf_prefill(ctypes.byref(p), n, _ptr(q), _ptr(k), _ptr(v), sb, sh, st, _ptr(out),
                                _ptr(scores), _ptr(kept_idx), _ptr(lse), _ptr(workspace),
                                workspace.numel(), _stream(stream)), "a2sf_prefill")
    else:
        assert alphas.dtype == torch.float32 and alphas.is_contiguous() and alphas.numel() == B * H
        _check(lib.a2sf_prefill_per_head(ctypes.byref(p), n, _ptr(q), _ptr(k), _ptr(v), sb, sh, st,
                                         _ptr(alphas), _ptr(out), _ptr(scores), _ptr(kept_idx), _ptr(lse),
                                         _ptr(workspace), workspace.numel(), _stream(stream)),
               "a2sf_prefill_per_head")
    return out, scores, kept_idx, lse


def a2sf_prefill_group(p: a2sf_params, group: int, q, k, v, stream=None):
    """Grouped query heads: q [B, H*group, n, d], k, v [B, H, n, d] (p.H = K/V heads).
    Returns (out [B,H*group,n,d], scores [B,H,n], kept_idx [B,H,m], lse [B,H*group,n])."""
    B, Hq, n, d = q.shape
    assert Hq == p.H * group and k.shape == (B, p.H, n, d) and v.shape == k.shape
    assert _strides(v) == _strides(k)
    dev = q.device
    out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=dev)
    scores = torch.empty((B, p.H, n), dtype=torch.float32, device=dev)
    kept = torch.empty((B, p.H, min(n, p.budget)), dtype=torch.int32, device=dev)
    lse = torch.empty((B, Hq, n), dtype=torch.float32, device=dev)
    nbytes = int(lib.a2sf_prefill_group_workspace_bytes(ctypes.byref(p), group, n))
    if nbytes == 0:
        raise A2SFError(A2SF_ERR_INVALID_ARG, "a2sf_prefill_group_workspace_bytes")
    ws = torch.empty((nbytes,), dtype=torch.uint8, device=dev)
    _check(lib.a2sf_prefill_group(ctypes.byref(p), group, n, _ptr(q), *_strides(q), _ptr(k), _ptr(v),
                                  *_strides(k), _ptr(out), _ptr(scores), _ptr(kept), _ptr(lse), _ptr(ws),
                                  nbytes, _stream(stream)), "a2sf_prefill_group")
    return out, scores, kept, lse


def a2sf_rescore(p: a2sf_params, q, k, lse, scores=None, kept_idx=None, workspace=None,
                 stream=None, alphas=None):
    """Scores and kept set for ``p.alpha`` from an existing log-sum-exp."""
    B, H, n, d = q.shape
    dev = q.device
    m = min(n, p.budget)
    scores = torch.empty((B, H, n), dtype=torch.float32, device=dev) if scores is None else scores
    kept_idx = torch.empty((B, H, m), dtype=torch.int32, device=dev) if kept_idx is None else kept_idx
    sb, sh, st = _strides(q)
    assert _strides(k) == (sb, sh, st)
    if workspace is None:
        need = a2sf_rescore_workspace_bytes(p, n)
        workspace = torch.empty((need,), dtype=torch.uint8, device=dev) if need else None
    wsn = workspace.numel() if workspace is not None else 0
    if alphas is None:
        _check(lib.a2sf_rescore(ctypes.byref(p), n, _ptr(q), _ptr(k), sb, sh, st, _ptr(lse),
                                _ptr(scores), _ptr(kept_idx), _ptr(workspace), wsn,
                                _stream(stream)), "a2sf_rescore")
    else:
        assert alphas.dtype == torch.float32 and alphas.is_contiguous() and alphas.numel() == B * H
        _check(lib.a2sf_rescore_per_head(ctypes.byref(p), n, _ptr(q), _ptr(k), sb, sh, st, _ptr(lse),
                                         _ptr(alphas), _ptr(scores), _ptr(kept_idx), _ptr(workspace), wsn,
                                         _stream(stream)), "a2sf_rescore_per_head")
    return scores, kept_idx


def a2sf_prefill_static_scratch(p: a2sf_params, q, k, v, out, scores, kept_idx, stream=None):
    """Prefill for callers that cannot allocate: every tensor is supplied by the
    caller and the library's built-in scratch array is used (size limit: see
    ``a2sf_prefill_static_scratch_max_rows``).  Returns the status code."""
    sb, sh, st = _strides(q)
    return int(lib.a2sf_prefill_static_scratch(ctypes.byref(p), q.shape[2], _ptr(q), _ptr(k), _ptr(v),
                                               sb, sh, st, _ptr(out), _ptr(scores), _ptr(kept_idx),
                                               _stream(stream)))


def a2sf_prefill_host_workspace_bytes(p: a2sf_params, n: int) -> int:
    return int(lib.a2sf_prefill_host_workspace_bytes(ctypes.byref(p), n))


def a2sf_prefill_host(p: a2sf_params, n: int, q_host, k_host, v_host, out_host, scores_host,
                      kept_host, workspace, stream=None):
    """Host-buffer prefill.  Returns the device addresses (ints) of k, v, scores,
    kept_idx inside ``workspace`` for a following ``a2sf_cache_load``."""
    dk, dv, ds, dkept = (ctypes.c_void_p() for _ in range(4))
    _check(lib.a2sf_prefill_host(ctypes.byref(p), n, _ptr(q_host), _ptr(k_host), _ptr(v_host),
                                 _ptr(out_host), _ptr(scores_host), _ptr(kept_host),
                                 _ptr(workspace), workspace.numel(), ctypes.byref(dk),
                                 ctypes.byref(dv), ctypes.byref(ds), ctypes.byref(dkept),
                                 _stream(stream)), "a2sf_prefill_host")
    return dk.value, dv.value, ds.value, dkept.value


class Cache:
    """Owner of an ``a2sf_cache`` whose storage is a torch device buffer."""

    def __init__(self, p: a2sf_params, device="cuda"):
        self.p = p
        self.bytes = int(lib.a2sf_cache_bytes(ctypes.byref(p)))
        if self.bytes == 0:
            raise A2SFError(A2SF_ERR_INVALID_ARG, "a2sf_cache_bytes")
        self.mem = torch.empty((self.bytes,), dtype=torch.uint8, device=device)
        h = ctypes.c_void_p()
        _check(lib.a2sf_cache_create(ctypes.byref(p), _ptr(self.mem), self.bytes, ctypes.byref(h)),
               "a2sf_cache_create")
        self.handle = h
        self.U, self.M, self.d = p.B * p.H, p.budget, p.d
        self.torch_dtype = {v: k for k, v in _DTYPE_CODE.items()}[p.dtype]

    def close(self):
        if getattr(self, "handle", None) and lib is not None:   # lib is None at interpreter exit
            lib.a2sf_cache_destroy(self.handle)
            self.handle = None

    __del__ = close

    def a2sf_cache_load(self, k, v, scores, kept_idx, n=None, strides=None, stream=None):
        """k, v: device tensors [B,H,n,d] (or raw addresses with ``n`` and ``strides``)."""
        if isinstance(k, torch.Tensor):
            n = k.shape[2]
            strides = _strides(k)
        sb, sh, st = strides
        _check(lib.a2sf_cache_load(self.handle, n, _ptr(k), _ptr(v), sb, sh, st, _ptr(scores),
                                   _ptr(kept_idx), _stream(stream)), "a2sf_cache_load")

    def a2sf_decode_step(self, alpha, q, k_new, v_new, out, evicted, stream=None):
        _check(lib.a2sf_decode_step(self.handle, alpha, _ptr(q), _ptr(k_new), _ptr(v_new),
                                    _ptr(out), _ptr(evicted), _stream(stream)), "a2sf_decode_step")

    def a2sf_decode_step_per_head(self, alphas, q, k_new, v_new, out, evicted, stream=None):
        """``alphas``: device tensor [B,H] fp32, one forgetting factor per unit."""
        assert alphas.dtype == torch.float32 and alphas.is_contiguous() and alphas.numel() == self.U
        _check(lib.a2sf_decode_step_per_head(self.handle, _ptr(alphas), _ptr(q), _ptr(k_new), _ptr(v_new),
                                             _ptr(out), _ptr(evicted), _stream(stream)),
               "a2sf_decode_step_per_head")

    def a2sf_decode_step_group(self, group, alpha, q, k_new, v_new, out, evicted, stream=None):
        """q, out [B, H*group, d]; k_new, v_new [B, H, d]; evicted [B, H]."""
        assert q.is_contiguous() and out.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous()
        _check(lib.a2sf_decode_step_group(self.handle, group, alpha, _ptr(q), _ptr(k_new), _ptr(v_new),
                                          _ptr(out), _ptr(evicted), _stream(stream)),
               "a2sf_decode_step_group")

    def a2sf_decode_step_host(self, alpha, q, k_new, v_new, out, evicted, stream=None):
        _check(lib.a2sf_decode_step_host(self.handle, alpha, _ptr(q), _ptr(k_new), _ptr(v_new),
                                         _ptr(out), _ptr(evicted), _stream(stream)),
               "a2sf_decode_step_host")

    def a2sf_cache_reset(self, stream=None):
        _check(lib.a2sf_cache_reset(self.handle, _stream(stream)), "a2sf_cache_reset")

    def a2sf_decode_multi(self, alpha, q, k_new, v_new, out=None, evicted=None, stream=None):
        """Appends the tokens of q, k_new, v_new [B,H,steps,d] one after the other."""
        return self._token_rows(lib.a2sf_decode_multi, "a2sf_decode_multi", alpha, q, k_new, v_new,
                                out, evicted, stream)

    def a2sf_prefill_streaming(self, alpha, q, k, v, out=None, evicted=None, stream=None):
        """Prunes while the prompt is processed: q, k, v [B,H,n,d] (one stride set).  Returns
        (out [B,H,n,d], evicted [n,B,H] int32)."""
        return self._token_rows(lib.a2sf_prefill_streaming, "a2sf_prefill_streaming", alpha, q, k, v,
                                out, evicted, stream)

    def a2sf_ideal_similarity(self, alpha, q, k, v, stream=None):
        """Streams the prompt through the policy and returns (cos [B,H,n] fp32, out, evicted):
        per row, the cosine between the policy's attention and the ideal top-(budget+1) row."""
        B, H, n, d = q.shape
        assert (B, H, d) == (self.p.B, self.p.H, self.d) and q.dtype == self.torch_dtype
        assert _strides(k) == _strides(q) and _strides(v) == _strides(q)
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
        ev = torch.empty((n, B, H), dtype=torch.int32, device=q.device)
        cos = torch.empty((B, H, n), dtype=torch.float32, device=q.device)
        nbytes = int(lib.a2sf_ideal_similarity_workspace_bytes(ctypes.byref(self.p), n))
        if nbytes == 0:
            raise A2SFError(A2SF_ERR_INVALID_ARG, "a2sf_ideal_similarity_workspace_bytes")
        ws = torch.empty((nbytes,), dtype=torch.uint8, device=q.device)
        sb, sh, st = _strides(q)
        _check(lib.a2sf_ideal_similarity(self.handle, alpha, n, _ptr(q), _ptr(k), _ptr(v), sb, sh, st,
                                         _ptr(out), _ptr(cos), _ptr(ev), _ptr(ws), nbytes,
                                         _stream(stream)), "a2sf_ideal_similarity")
        return cos, out, ev

    def _token_rows(self, fn, name, alpha, q, k, v, out, evicted, stream):
        B, H, n, d = q.shape
        assert (B, H, d) == (self.p.B, self.p.H, self.d) and q.dtype == self.torch_dtype
        assert k.shape == q.shape and v.shape == q.shape
        assert _strides(k) == _strides(q) and _strides(v) == _strides(q)
        if out is None:
            out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
        assert _strides(out) == _strides(q)
        if evicted is None:
            evicted = torch.empty((n, B, H), dtype=torch.int32, device=q.device)
        sb, sh, st = _strides(q)
        _check(fn(self.handle, alpha, n, _ptr(q), _ptr(k), _ptr(v), sb, sh, st,
                  _ptr(out), _ptr(evicted), _stream(stream)), name)
        return out, evicted

    def state_tensors(self, device=None):
        device = device or self.mem.device
        B, H, M, d = self.p.B, self.p.H, self.M, self.d
        return {
            "k": torch.empty((B, H, M, d), dtype=self.torch_dtype, device=device),
            "v": torch.empty((B, H, M, d), dtype=self.torch_dtype, device=device),
            "scores": torch.empty((B, H, M), dtype=torch.float32, device=device),
            "pos": torch.empty((B, H, M), dtype=torch.int32, device=device),
            "count": torch.empty((B, H), dtype=torch.int32, device=device),
            "len": torch.empty((B, H), dtype=torch.int32, device=device),
        }

    def a2sf_cache_export(self, state=None, stream=None):
        state = state or self.state_tensors()
        _check(lib.a2sf_cache_export(self.handle, *(_ptr(state.get(k)) for k in
                                                    ("k", "v", "scores", "pos", "count", "len")),
                                     _stream(stream)), "a2sf_cache_export")
        return state

    def a2sf_cache_import(self, state, stream=None):
        _check(lib.a2sf_cache_import(self.handle, *(_ptr(state.get(k)) for k in
                                                    ("k", "v", "scores", "pos", "count", "len")),
                                     _stream(stream)), "a2sf_cache_import")
