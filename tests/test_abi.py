"""The C ABI without a GPU: the library loads, exports what the header declares and
rejects bad arguments on the host before anything is launched."""
import ctypes
import re

import numpy as np
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def a2sf():
    from paper_2407_20485_b200 import build

    build.build()
    from paper_2407_20485_b200 import binding

    return binding


def _declared_functions():
    text = (ROOT / "include" / "a2sf.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(a2sf_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(a2sf):
    names = _declared_functions()
    assert "a2sf_prefill" in names and "a2sf_decode_step" in names and len(names) >= 17
    raw = ctypes.CDLL(str(ROOT / "paper_2407_20485_b200" / "liba2sf.so"))
    for name in names:
        assert hasattr(raw, name), f"{name} declared in a2sf.h but not exported"
    assert sorted(a2sf.EXPORTED) == names


def test_status_strings(a2sf):
    assert a2sf.status_string(0) == "ok"
    for code in (-1, -2, -3, -4, -5):
        assert a2sf.status_string(code) not in ("ok", "unknown status")
    assert a2sf.status_string(-99) == "unknown status"


def test_size_queries_need_no_gpu(a2sf):
    import torch

    p = a2sf.make_params(32, 40, 128, torch.bfloat16, 512, 256, 0.5)
    U, M, d = 1280, 512, 128
    assert a2sf.a2sf_prefill_workspace_bytes(p, 4096) >= U * 4096 * 4
    cache_bytes = a2sf.lib.a2sf_cache_bytes(ctypes.byref(p))
    assert cache_bytes >= 2 * U * M * d * 2 + 2 * U * M * 4 + 2 * U * 4
    assert cache_bytes % 256 == 0
    assert a2sf.a2sf_prefill_host_workspace_bytes(p, 4096) > 4 * U * 4096 * d * 2


@pytest.mark.parametrize("field,value,status", [
    ("d", 96, -2), ("dtype", 7, -2), ("budget", 0, -1), ("recent", 600, -1), ("recent", -1, -1),
    ("alpha", 1.5, -1), ("alpha", -0.1, -1), ("alpha", float("nan"), -1), ("B", 0, -1),
    ("scale", -1.0, -1), ("flags", 8, -1),
])
def test_bad_parameters_are_rejected_on_the_host(a2sf, field, value, status):
    import torch

    p = a2sf.make_params(1, 2, 128, torch.bfloat16, 512, 256, 0.5)
    setattr(p, field, value)
    assert a2sf.a2sf_prefill_workspace_bytes(p, 128) == 0
    assert a2sf.lib.a2sf_cache_bytes(ctypes.byref(p)) == 0
    h = ctypes.c_void_p()
    assert a2sf.lib.a2sf_cache_create(ctypes.byref(p), None, 0, ctypes.byref(h)) == status
    fake = ctypes.c_void_p(0x1000)
    rc = a2sf.lib.a2sf_prefill(ctypes.byref(p), 128, fake, fake, fake, 128 * 256, 128 * 128, 128,
                               fake, fake, fake, None, fake, 1 << 30, None)
    assert rc == status


def test_bad_pointers_and_strides_are_rejected_on_the_host(a2sf):
    import torch

    p = a2sf.make_params(1, 2, 128, torch.bfloat16, 512, 256, 0.5)
    ok = ctypes.c_void_p(0x10000)
    odd = ctypes.c_void_p(0x10008)
    call = a2sf.lib.a2sf_prefill
    base = dict(n=128, sb=2 * 128 * 128, sh=128 * 128, st=128)

    def prefill(q=ok, k=ok, v=ok, out=ok, scores=ok, kept=ok, ws=ok, ws_bytes=1 << 30, **o):
        a = {**base, **o}
        return call(ctypes.byref(p), a["n"], q, k, v, a["sb"], a["sh"], a["st"], out, scores, kept,
                    None, ws, ws_bytes, None)

    assert prefill(q=None) == a2sf.A2SF_ERR_INVALID_ARG
    assert prefill(kept=None) == a2sf.A2SF_ERR_INVALID_ARG
    assert prefill(k=odd) == a2sf.A2SF_ERR_INVALID_ARG           # rows must be 16-byte aligned
    assert prefill(st=100) == a2sf.A2SF_ERR_INVALID_ARG          # token stride below d
    assert prefill(st=132) == a2sf.A2SF_ERR_INVALID_ARG          # stride not a multiple of 16 bytes
    assert prefill(n=0) == a2sf.A2SF_ERR_INVALID_ARG
    assert prefill(ws=None) == a2sf.A2SF_ERR_INVALID_ARG
    assert prefill(ws_bytes=16) == a2sf.A2SF_ERR_WORKSPACE
    assert a2sf.lib.a2sf_decode_step(None, 0.5, ok, ok, ok, ok, ok, None) == a2sf.A2SF_ERR_INVALID_ARG
    assert a2sf.lib.a2sf_cache_destroy(None) == a2sf.A2SF_ERR_INVALID_ARG
    assert a2sf.lib.a2sf_cache_load(None, 8, ok, ok, 1, 1, 1, ok, ok, None) == a2sf.A2SF_ERR_INVALID_ARG


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    import importlib
    import sys

    from paper_2407_20485_b200 import binding

    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "liba2sf.so")
    with pytest.raises(ImportError, match="no CPU fallback"):
        binding._load()


def test_score_window_bound_is_the_tail_of_the_geometric_series():
    """Host arithmetic only: the bound equals the summed weights of the rows left out."""
    from paper_2407_20485_b200 import binding as a2sf

    for alpha, n, Wn in [(0.5, 100, 10), (0.9, 4096, 200), (1.0, 50, 20), (0.0, 30, 3), (0.3, 10, 10),
                         (0.7, 10, 0), (0.99, 500, 499)]:
        # fp32 alpha, as the library receives it
        a = float(np.float32(alpha))
        tail = sum(a ** age for age in range(Wn, n)) if 0 < Wn < n else 0.0
        got = a2sf.a2sf_score_window_bound(alpha, n, Wn)
        assert abs(got - tail) <= 1e-12 * max(1.0, tail), (alpha, n, Wn, got, tail)


def test_budget_beyond_the_documented_maximum_is_refused_on_the_host():
    import torch
    from paper_2407_20485_b200 import binding as a2sf

    ok = a2sf.make_params(1, 1, 128, torch.bfloat16, 49152, 16, 0.5)
    too_big = a2sf.make_params(1, 1, 128, torch.bfloat16, 49153, 16, 0.5)
    assert a2sf.lib.a2sf_cache_bytes(ctypes.byref(ok)) > 0
    assert a2sf.lib.a2sf_cache_bytes(ctypes.byref(too_big)) == 0
    assert a2sf.lib.a2sf_prefill_workspace_bytes(ctypes.byref(too_big), 64) == 0


def test_header_is_plain_c_and_links_from_a_c_program(tmp_path):
    """include/a2sf.h compiled as strict C99 by gcc, linked against the library, and a few
    host-only entry points called from C: no C++ or torch types at the boundary."""
    import subprocess

    from paper_2407_20485_b200 import binding

    root = Path(__file__).resolve().parents[1]
    src = tmp_path / "use_a2sf.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "a2sf.h"
int main(void)
{
    a2sf_params p;
    memset(&p, 0, sizeof p);
    p.B = 2; p.H = 4; p.d = 128; p.dtype = A2SF_BF16; p.budget = 64; p.recent = 32; p.alpha = 0.5f;
    if (a2sf_cache_bytes(&p) == 0) return 1;
    if (a2sf_prefill_workspace_bytes(&p, 300) == 0) return 2;
    p.recent = 65;                                     /* recent > budget */
    if (a2sf_cache_bytes(&p) != 0) return 3;
    if (a2sf_decode_step(NULL, 0.5f, NULL, NULL, NULL, NULL, NULL, NULL) != A2SF_ERR_INVALID_ARG) return 4;
    if (a2sf_score_window_bound(0.5f, 100, 3) <= 0.0) return 5;
    printf("%s\n", a2sf_status_string(A2SF_ERR_WORKSPACE));
    return 0;
}
''')
    exe = tmp_path / "use_a2sf"
    lib_dir = Path(binding._LIB_PATH).parent
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", str(root / "include"),
                    str(src), "-o", str(exe), f"-L{lib_dir}", "-la2sf", f"-Wl,-rpath,{lib_dir}"], check=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, (r.returncode, r.stdout, r.stderr)
    assert len(r.stdout.strip()) > 0
