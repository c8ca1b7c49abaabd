"""Argument checks of the C ABI that run on the host before any CUDA call: they need no GPU.
Every refusal is a return code (no exception crosses the boundary, nothing is launched)."""
import ctypes

import pytest
import torch

from paper_2407_20485_b200 import binding as a2sf

OK, INVALID, UNSUPPORTED, WORKSPACE = 0, -1, -2, -5
FAKE = ctypes.c_void_p(0x1000)          # a 256-byte aligned non-null address that is never dereferenced


def _p(**kw):
    base = dict(B=1, H=2, d=128, dtype=torch.bfloat16, budget=64, recent=32, alpha=0.5)
    base.update(kw)
    return a2sf.make_params(**base)


def _prefill(p, n=256, q=FAKE, k=FAKE, v=FAKE, strides=None, out=FAKE, scores=FAKE, kept=FAKE, ws=FAKE,
             ws_bytes=1 << 40):
    sb, sh, st = strides or (p.H * n * p.d, n * p.d, p.d)
    return a2sf.lib.a2sf_prefill(ctypes.byref(p), n, q, k, v, sb, sh, st, out, scores, kept, None, ws,
                                 ws_bytes, None)


@pytest.mark.parametrize("kw,want", [
    (dict(B=0), INVALID), (dict(H=0), INVALID), (dict(budget=0), INVALID),
    (dict(recent=-1), INVALID), (dict(recent=65), INVALID),
    (dict(alpha=-0.1), INVALID), (dict(alpha=1.5), INVALID), (dict(alpha=float("nan")), INVALID),
    (dict(scale=-1.0), INVALID), (dict(scale=float("inf")), INVALID),
    (dict(d=96), UNSUPPORTED), (dict(budget=49153, recent=0), UNSUPPORTED),
    (dict(flags=2), INVALID), (dict(score_window=-1), INVALID),
])
def test_parameter_block_is_checked(kw, want):
    p = _p(**kw)
    assert _prefill(p) == want
    assert a2sf.lib.a2sf_prefill_workspace_bytes(ctypes.byref(p), 256) == 0
    assert a2sf.lib.a2sf_cache_bytes(ctypes.byref(p)) == 0


def test_dtype_outside_the_enumeration_is_unsupported():
    p = _p()
    p.dtype = 7
    assert _prefill(p) == UNSUPPORTED


def test_prefill_pointer_stride_and_workspace_checks():
    p = _p()
    assert _prefill(p, n=0) == INVALID
    for name in ("q", "k", "v", "out", "scores", "kept", "ws"):
        assert _prefill(p, **{name: None}) == INVALID, name
    assert _prefill(p, q=ctypes.c_void_p(0x1008)) == INVALID              # rows must be 16-byte aligned
    assert _prefill(p, ws=ctypes.c_void_p(0x1010)) == INVALID             # workspace 256-byte aligned
    assert _prefill(p, strides=(2 * 256 * 128, 256 * 128, 64)) == INVALID   # token stride below d
    assert _prefill(p, strides=(2 * 256 * 128, 256 * 128 + 4, 128)) == INVALID   # stride not a multiple of 16 bytes
    need = a2sf.lib.a2sf_prefill_workspace_bytes(ctypes.byref(p), 256)
    assert need > 0 and _prefill(p, ws_bytes=need - 1) == WORKSPACE


def test_grouped_prefill_checks():
    p = _p()
    f = a2sf.lib.a2sf_prefill_group
    n = 128
    args = lambda group, pp=p: (ctypes.byref(pp), group, n, FAKE, 4 * n * 128, n * 128, 128, FAKE, FAKE,
                                2 * n * 128, n * 128, 128, FAKE, FAKE, FAKE, None, FAKE, 1 << 40, None)
    assert f(*args(0)) == UNSUPPORTED and f(*args(9)) == UNSUPPORTED
    assert f(*args(2, _p(score_window=8))) == UNSUPPORTED
    assert a2sf.lib.a2sf_prefill_group_workspace_bytes(ctypes.byref(p), 9, n) == 0
    assert a2sf.lib.a2sf_prefill_group_workspace_bytes(ctypes.byref(p), 4, n) > 0


def test_null_cache_and_size_queries():
    lib = a2sf.lib
    assert lib.a2sf_decode_step(None, 0.5, FAKE, FAKE, FAKE, FAKE, FAKE, None) == INVALID
    assert lib.a2sf_decode_step_group(None, 2, 0.5, FAKE, FAKE, FAKE, FAKE, FAKE, None) == INVALID
    assert lib.a2sf_decode_multi(None, 0.5, 4, FAKE, FAKE, FAKE, 1, 1, 128, FAKE, None, None) == INVALID
    assert lib.a2sf_prefill_streaming(None, 0.5, 4, FAKE, FAKE, FAKE, 1, 1, 128, FAKE, None, None) == INVALID
    assert lib.a2sf_cache_reset(None, None) == INVALID
    assert lib.a2sf_cache_destroy(None) == INVALID
    p = _p()
    assert lib.a2sf_ideal_similarity_workspace_bytes(ctypes.byref(p), 32769) == 0
    assert lib.a2sf_ideal_similarity_workspace_bytes(ctypes.byref(p), 1024) >= 2 * 1024 * 16
    assert lib.a2sf_prefill_static_scratch_max_rows() == 1 << 20
    assert lib.a2sf_select(ctypes.byref(p), 0, FAKE, FAKE, None) == INVALID
    assert lib.a2sf_select(ctypes.byref(p), 64, None, FAKE, None) == INVALID
    assert lib.a2sf_select(ctypes.byref(_p(budget=0)), 64, FAKE, FAKE, None) == INVALID
    # the bounded-wait self-test refuses anything that is not a short, bounded wait before any CUDA call
    for which, limit, rep in ((2, 1000, FAKE), (-1, 1000, FAKE), (0, 0, FAKE), (0, 2_000_000_001, FAKE),
                              (1, 1000, None), (1, 1000, ctypes.c_void_p(0x1004))):
        assert lib.a2sf_selftest_bounded_wait(which, limit, rep, None) == INVALID
    for code in (0, -1, -2, -3, -4, -5, 99):
        assert len(lib.a2sf_status_string(code)) > 0
