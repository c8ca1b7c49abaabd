"""The small-shape sweep under the bounds-checked library, with canary words around every buffer.

compute-sanitizer is not available where this suite runs, so the library has a build of its own
(-DA2SF_DEBUG, liba2sf_debug.so) in which every slot, position, tile-row and ring-stage index that
addresses memory inside a kernel is range-checked and reported instead of used, and the harness
can put guard regions around all the device memory it hands to the library.  The sweep runs in a
child process because the library is chosen when the binding is imported.
"""
import os
import subprocess
import sys
from pathlib import Path

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent
SWEEP = ("tiny_fp32_full or shrunken_configs or edge_cases or random_shapes or grouped_query_heads or "
         "streamed_prompt or per_head_forgetting or similarity_with_the_ideal or several_tokens or "
         "truncated_scoring or zero_weight_rows or late_dominant or values_beyond_fp16 or selection_alone")


def test_small_shape_sweep_under_the_bounds_checked_library_with_guard_words():
    from paper_2407_20485_b200 import build

    build.build(debug=True)          # incremental: a no-op when liba2sf_debug.so is up to date
    assert build.DEBUG_LIB_PATH.exists()
    env = dict(os.environ, A2SF_LIBRARY="debug", A2SF_GUARDS="1")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_parity_gpu.py", "-k", SWEEP]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    line = [x for x in r.stdout.splitlines() if x.startswith("[debug sweep]")]
    assert line, tail
    print(line[0])
    from conftest import report_line

    report_line(line[0])
    assert " 0 index violations" in line[0]
    ntests = int(line[0].split()[2])
    assert ntests >= 60, line[0]


def test_the_release_library_reports_no_debug_record():
    from paper_2407_20485_b200 import binding as a2sf

    if os.environ.get("A2SF_LIBRARY", "") == "debug":
        pytest.skip("this process runs the debug library")
    assert not a2sf.a2sf_debug_build()
    assert a2sf.a2sf_debug_violations() == (0, 0, 0, 0, 0)


def test_the_debug_library_reports_an_out_of_range_index_and_skips_nothing_it_should_not():
    """Positive control, in a child process: a kept index beyond the prompt is input that the cache
    build already clamps; the bounds-checked library must also report it, with its value and bound."""
    code = r'''
import torch
from paper_2407_20485_b200 import binding as a2sf, workloads as wl
assert a2sf.a2sf_debug_build()
w = wl.WORKLOADS["llama2_7b"].scaled(H=2, n=200, budget=32, recent=16, steps=0)
q, k, v = wl.make_prompt(w, device="cuda")
p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha)
_, S, kept, _ = a2sf.a2sf_prefill(p, q, k, v)
torch.cuda.synchronize()
assert a2sf.a2sf_debug_violations()[0] == 0
bad = kept.clone()
bad[0, 1, 5] = w.n + 7
cache = a2sf.Cache(p)
cache.a2sf_cache_load(k, v, S, bad)
torch.cuda.synchronize()
count, kernel, line, index, bound = a2sf.a2sf_debug_violations()
assert count == 32 and index == w.n + 7          # every lane of the slot's warp sees the index
assert bound == w.n and kernel == 2, (count, kernel, line, index, bound)
assert a2sf.a2sf_debug_violations()[0] == 0          # cleared by the read
st = cache.a2sf_cache_export()
torch.cuda.synchronize()
assert int(st["pos"][0, 1, 5]) == w.n - 1            # clamped into the prompt, as in the release library
print("positive control ok")
'''
    from paper_2407_20485_b200 import build

    build.build(debug=True)
    env = dict(os.environ, A2SF_LIBRARY="debug")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "positive control ok" in r.stdout, r.stdout[-2000:] + r.stderr[-3000:]


def test_guard_words_catch_a_write_outside_the_buffer():
    """The guard check itself, with the stray write made from the host side (torch), not by a kernel."""
    from guards import GUARD_BYTES, GuardedTorch

    g = GuardedTorch(torch)
    t = g.empty((3, 5), dtype=torch.float32, device="cuda")
    s = g.empty_strided((2, 2, 4, 8), (80, 40, 10, 1), dtype=torch.bfloat16, device="cuda")
    assert t.shape == (3, 5) and s.stride() == (80, 40, 10, 1) and t.data_ptr() % 256 == 0
    t.fill_(1.0)
    s.fill_(2.0)
    g.check("clean")
    base, nbytes = g._bases[0]
    base[GUARD_BYTES + nbytes + 3] = 0          # one byte past the end of t
    with pytest.raises(AssertionError, match="wrote outside"):
        g.check("dirty")
