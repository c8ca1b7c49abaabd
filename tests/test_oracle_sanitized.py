"""The C oracle under AddressSanitizer and UndefinedBehaviorSanitizer (host code only).

The oracle is what every parity claim rests on, so its own memory accesses are checked too: a
sanitized build of ``oracle/a2sf_oracle.c`` runs a prefill with selection, a cache build and a run
of generation steps with evictions (several threads, ragged sizes, budget 1, no recent window) in a
child process; any out-of-bounds access, use after free or undefined operation aborts it.
"""
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

CODE = r'''
import sys
import numpy as np
sys.path.insert(0, %(root)r)
import oracle
lib = oracle.load(%(lib)r)
rng = np.random.default_rng(7)
for (U, n, d, M, R, T, alphas) in ((3, 37, 8, 9, 4, 25, [0.5, 0.0, 1.0]), (2, 5, 16, 1, 0, 12, [0.3]),
                                   (1, 1, 4, 4, 4, 6, [1.0]), (4, 64, 32, 16, 16, 20, [0.9])):
    Q, K, V = (rng.standard_normal((U, n, d)) for _ in range(3))
    ref = oracle.prefill(Q, K, V, 1.0 / np.sqrt(d), alphas, M, R, nthreads=3, lib=lib)
    assert ref["out"].shape == (U, n, d) and np.isfinite(ref["S"]).all()
    assert abs(ref["S"][:, 0].sum(axis=1) - sum(alphas[0] ** a for a in range(n))).max() < 1e-9
    cache = oracle.Cache(U, d, M, R, 1.0 / np.sqrt(d), lib=lib)
    cache.load(K, V, ref["S"][:, 0], ref["kept"])
    for t in range(T):
        q, k, v = (rng.standard_normal((U, d)) for _ in range(3))
        out, info, sc = cache.step(q, k, v, alphas[0], nthreads=2)
        assert np.isfinite(out).all()
    assert (cache.count == min(n + T, M)).all() and (cache.len == n + T).all()
print("sanitized oracle ok")
'''


def test_oracle_runs_clean_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    import oracle

    asan = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    if not asan or not Path(asan).exists():
        pytest.skip("gcc has no libasan here")
    lib = tmp_path / "liba2sf_oracle_san.so"
    oracle.build(force=True, out=lib,
                 extra_cflags=["-g", "-O1", "-fno-omit-frame-pointer", "-fsanitize=address,undefined",
                               "-fno-sanitize-recover=undefined"])
    env = dict(os.environ, LD_PRELOAD=asan, ASAN_OPTIONS="detect_leaks=0:abort_on_error=1",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    r = subprocess.run([sys.executable, "-c", CODE % {"root": str(ROOT), "lib": str(lib)}],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "sanitized oracle ok" in r.stdout, (r.stdout[-1500:] + r.stderr[-3000:])
