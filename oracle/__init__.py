"""ctypes front end of the fp64 CPU oracle (``a2sf_oracle.c``).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's CPU-baseline
leg import this package.  It shares no code with the CUDA library and never
imports it.  All arrays are numpy float64 / int32, C-contiguous.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path
from typing import Optional, Sequence

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "a2sf_oracle.c"
_LIB_PATH = _HERE / "liba2sf_oracle.so"
_lib = None

_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False, extra_cflags: Sequence[str] = (), out: Optional[Path] = None) -> Path:
    """Compile the oracle with gcc (plain -O2, no fast-math: fp64 as written)."""
    out = Path(out) if out else _LIB_PATH
    if not force and out.exists() and out.stat().st_mtime >= _SRC.stat().st_mtime:
        return out
    tmp = out.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O2", "-fPIC", "-shared", "-std=c11", "-pthread", *extra_cflags,
           str(_SRC), "-o", str(tmp), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


def _bind(lib):
    c_int, c_dbl = ctypes.c_int, ctypes.c_double
    lib.a2sf_oracle_softmax_row.restype = c_dbl
    lib.a2sf_oracle_softmax_row.argtypes = [_D, _D, c_int, c_dbl, c_int, _D]
    lib.a2sf_oracle_prefill_rows.restype = None
    lib.a2sf_oracle_prefill_rows.argtypes = [_D, _D, _D, c_int, c_int, c_dbl, _D, c_int,
                                             c_int, c_int, _D, _D, _D]
    lib.a2sf_oracle_select.restype = c_int
    lib.a2sf_oracle_select.argtypes = [_D, c_int, c_int, c_int, _I]
    lib.a2sf_oracle_cache_load.restype = None
    lib.a2sf_oracle_cache_load.argtypes = [_D, _D, _D, _I, c_int, c_int, c_int,
                                           _D, _D, _D, _I, _I, _I]
    lib.a2sf_oracle_decode_step.restype = None
    lib.a2sf_oracle_decode_step.argtypes = [_D, _D, _D, _I, _I, _I, _D, _D, _D,
                                            c_int, c_dbl, c_dbl, c_int, c_int, c_int,
                                            _D, _I, _D]
    lib.a2sf_oracle_prefill_batch.restype = c_int
    lib.a2sf_oracle_prefill_batch.argtypes = [_D, _D, _D, c_int, c_int, c_int, c_dbl,
                                              _D, c_int, c_int, c_int, c_int,
                                              _D, _D, _D, _I, _I, c_int]
    lib.a2sf_oracle_decode_step_batch.restype = c_int
    lib.a2sf_oracle_decode_step_batch.argtypes = [_D, _D, _D, _I, _I, _I, _D, _D, _D,
                                                  c_int, c_int, c_dbl, c_dbl, c_int, c_int,
                                                  _I, _D, _I, _D, c_int]
    return lib


def load(path: Optional[Path] = None):
    """Load (building if needed) the oracle library."""
    global _lib
    if path is not None:
        return _bind(ctypes.CDLL(str(path)))
    if _lib is None:
        _lib = _bind(ctypes.CDLL(str(build())))
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _dp(a: Optional[np.ndarray]):
    return a.ctypes.data_as(_D) if a is not None else None


def _ip(a: Optional[np.ndarray]):
    return a.ctypes.data_as(_I) if a is not None else None


def host_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def attention_probs(Q, K, scale: float, lib=None) -> np.ndarray:
    """Materialised causal softmax matrix P [n, n] (tiny inputs only)."""
    lib = lib or load()
    Q, K = _f64(Q), _f64(K)
    n, d = Q.shape
    P = np.zeros((n, n), dtype=np.float64)
    for i in range(n):
        lib.a2sf_oracle_softmax_row(_dp(Q), _dp(K), d, float(scale), i, _dp(P[i]))
    return P


def prefill_rows(Q, K, V, scale: float, alphas: Sequence[float], i0: int, i1: int, lib=None):
    """Rows [i0, i1) of one unit: out rows, lse rows and their contribution to S."""
    lib = lib or load()
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, d = Q.shape
    al = _f64(list(alphas))
    out = np.empty((i1 - i0, d), dtype=np.float64)
    lse = np.empty((i1 - i0,), dtype=np.float64)
    S = np.empty((len(al), n), dtype=np.float64)
    lib.a2sf_oracle_prefill_rows(_dp(Q), _dp(K), _dp(V), n, d, float(scale), _dp(al), len(al),
                                 int(i0), int(i1), _dp(out), _dp(lse), _dp(S))
    return out, lse, S


def select(S, M: int, R: int, lib=None) -> np.ndarray:
    lib = lib or load()
    S = _f64(S)
    n = S.shape[0]
    kept = np.empty((min(n, M),), dtype=np.int32)
    m = lib.a2sf_oracle_select(_dp(S), n, int(M), int(R), _ip(kept))
    assert m == kept.shape[0]
    return kept


def prefill(Q, K, V, scale: float, alphas: Sequence[float], M: int, R: int,
            sel_alpha: int = 0, nthreads: int = 1, want_out: bool = True, lib=None):
    """Full prefill of U units.  Q, K, V: [U, n, d].  Returns a dict with
    out [U,n,d], lse [U,n], S [U,A,n], kept [U,min(n,M)] and the thread count used."""
    lib = lib or load()
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    U, n, d = Q.shape
    al = _f64(list(alphas))
    A = len(al)
    out = np.empty((U, n, d), dtype=np.float64) if want_out else None
    lse = np.empty((U, n), dtype=np.float64)
    S = np.empty((U, A, n), dtype=np.float64)
    m = min(n, M)
    kept = np.empty((U, m), dtype=np.int32)
    kept_len = np.empty((U,), dtype=np.int32)
    used = lib.a2sf_oracle_prefill_batch(_dp(Q), _dp(K), _dp(V), U, n, d, float(scale),
                                         _dp(al), A, int(M), int(R), int(sel_alpha),
                                         _dp(out), _dp(lse), _dp(S), _ip(kept), _ip(kept_len),
                                         int(nthreads))
    assert (kept_len == m).all()
    return {"out": out, "lse": lse, "S": S, "kept": kept, "threads": used}


class Cache:
    """Slot-indexed pruned cache of U units, stepped by the oracle."""

    def __init__(self, U: int, d: int, M: int, R: int, scale: float, lib=None):
        self.lib = lib or load()
        self.U, self.d, self.M, self.R, self.scale = U, d, M, R, float(scale)
        self.K = np.zeros((U, M, d), dtype=np.float64)
        self.V = np.zeros((U, M, d), dtype=np.float64)
        self.S = np.zeros((U, M), dtype=np.float64)
        self.pos = np.full((U, M), -1, dtype=np.int32)
        self.count = np.zeros((U,), dtype=np.int32)
        self.len = np.zeros((U,), dtype=np.int32)

    def load(self, K, V, S, kept):
        """K, V [U,n,d]; S [U,n]; kept [U,m]: slot s <- token kept[s]."""
        K, V, S = _f64(K), _f64(V), _f64(S)
        kept = np.ascontiguousarray(kept, dtype=np.int32)
        U, n, d = K.shape
        m = kept.shape[1]
        for u in range(U):
            self.lib.a2sf_oracle_cache_load(_dp(K[u]), _dp(V[u]), _dp(S[u]), _ip(kept[u]),
                                            m, n, d, _dp(self.K[u]), _dp(self.V[u]),
                                            _dp(self.S[u]), _ip(self.pos[u]),
                                            _ip(self.count[u:u + 1]), _ip(self.len[u:u + 1]))

    def step(self, q, k_new, v_new, alpha: float, force=None, nthreads: int = 1):
        """One generation step for all units.  q, k_new, v_new: [U, d].
        ``force`` [U] int32: slot to vacate instead of the rule's choice when the
        cache is full (-3 = follow the rule).  ``alpha`` may be a scalar or one value per
        unit.  Returns out [U,d], info [U,3]
        (vacated, rule's choice, rule's runner-up) and their scores [U,3]."""
        q, k_new, v_new = _f64(q), _f64(k_new), _f64(v_new)
        out = np.empty((self.U, self.d), dtype=np.float64)
        info = np.empty((self.U, 3), dtype=np.int32)
        sc2 = np.empty((self.U, 3), dtype=np.float64)
        f = None if force is None else np.ascontiguousarray(force, dtype=np.int32)
        if np.ndim(alpha) == 0:
            self.lib.a2sf_oracle_decode_step_batch(
                _dp(self.K), _dp(self.V), _dp(self.S), _ip(self.pos), _ip(self.count), _ip(self.len),
                _dp(q), _dp(k_new), _dp(v_new), self.U, self.d, self.scale, float(alpha),
                self.M, self.R, _ip(f), _dp(out), _ip(info), _dp(sc2), int(nthreads))
        else:
            # one forgetting factor per unit: the single-unit step, unit by unit
            assert len(alpha) == self.U
            for u in range(self.U):
                self.lib.a2sf_oracle_decode_step(
                    _dp(self.K[u]), _dp(self.V[u]), _dp(self.S[u]), _ip(self.pos[u]),
                    _ip(self.count[u:u + 1]), _ip(self.len[u:u + 1]), _dp(q[u]), _dp(k_new[u]),
                    _dp(v_new[u]), self.d, self.scale, float(alpha[u]), self.M, self.R,
                    -3 if f is None else int(f[u]), _dp(out[u]), _ip(info[u]), _dp(sc2[u]))
        return out, info, sc2

    def snapshot(self):
        return {k: getattr(self, k).copy() for k in ("K", "V", "S", "pos", "count", "len")}

    def restore(self, snap):
        for k, v in snap.items():
            getattr(self, k)[...] = v


def streaming_prefill(Q, K, V, scale: float, alpha, M: int, R: int, force=None, nthreads: int = 1,
                      lib=None):
    """The prompt pruned while it is processed, row by row (the reading of the paper's mask
    figures, Sec. 3.2 / 4.3): starting from an empty cache, token i is one generation step with
    (q_i, k_i, v_i).  Q, K, V: [U, n, d].  ``force`` [n, U] int32 (or None) overrides the rule's
    choice per step as in ``Cache.step``.  Returns (out [U,n,d], info [n,U,3], scores [n,U,3],
    cache)."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    U, n, d = Q.shape
    cache = Cache(U, d, M, R, scale, lib=lib)
    out = np.empty((U, n, d), dtype=np.float64)
    info = np.empty((n, U, 3), dtype=np.int32)
    sc = np.empty((n, U, 3), dtype=np.float64)
    for i in range(n):
        o, info[i], sc[i] = cache.step(Q[:, i], K[:, i], V[:, i], alpha,
                                        force=None if force is None else force[i], nthreads=nthreads)
        out[:, i] = o
    return out, info, sc, cache


def ideal_row(s_row: np.ndarray, keep: int) -> np.ndarray:
    """Ideal pruning of one attention row (Sec. 4.3): of the row's logits the ``keep`` largest
    stay (equal logits: the lower position first), the softmax runs over those alone.
    Returns the full-length probability vector (zeros where pruned)."""
    m = s_row.shape[0]
    order = np.lexsort((np.arange(m), -s_row))[:min(keep, m)]
    w = np.exp(s_row[order] - s_row[order].max())
    p = np.zeros(m)
    p[order] = w / w.sum()
    return p


def ideal_similarity(Q, K, V, scale: float, alpha, M: int, R: int, force=None, nthreads: int = 1,
                     lib=None):
    """Cosine similarity, row by row, between the attention a pruning policy actually uses while
    the prompt streams through it and the ideal row that keeps the same number of tokens
    (M cached + the token itself) by magnitude alone (Sec. 4.3, the similarity table).
    Q, K, V: [U, n, d].  Returns (cos [U, n], out, info, scores, cache) with the last four as in
    ``streaming_prefill``."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    U, n, d = Q.shape
    cache = Cache(U, d, M, R, scale, lib=lib)
    cos = np.empty((U, n), dtype=np.float64)
    out = np.empty((U, n, d), dtype=np.float64)
    info = np.empty((n, U, 3), dtype=np.int32)
    sc = np.empty((n, U, 3), dtype=np.float64)
    for i in range(n):
        for u in range(U):
            s_row = (K[u, :i + 1] @ Q[u, i]) * scale
            seen = np.append(cache.pos[u, :cache.count[u]], i)          # cached tokens + itself
            w = np.exp(s_row[seen] - s_row[seen].max())
            meth = np.zeros(i + 1)
            meth[seen] = w / w.sum()
            ideal = ideal_row(s_row, M + 1)
            cos[u, i] = (meth @ ideal) / np.sqrt((meth @ meth) * (ideal @ ideal))
        o, info[i], sc[i] = cache.step(Q[:, i], K[:, i], V[:, i], alpha,
                                        force=None if force is None else force[i], nthreads=nthreads)
        out[:, i] = o
    return cos, out, info, sc, cache


# ---- grouped query heads: G query heads share one K/V head and therefore one pruned cache ----------
# The paper scores a token per head (Sec. 2.2); with a shared K/V head there is one set of tokens
# to keep, and the reading taken here is that its score is the SUM of the group's attention
# probabilities, accumulated and forgotten as in Eq. 5.

def group_prefill(Q, K, V, scale: float, alpha: float, M: int, R: int, nthreads: int = 1, lib=None):
    """Q [U, G, n, d] (U = batch x K/V heads), K, V [U, n, d].  Dense causal attention per query
    head; S = sum over the group of each head's Eq. 5 scores; one selection per K/V head.
    Returns out [U,G,n,d], lse [U,G,n], S [U,n], kept [U,min(n,M)]."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    U, G, n, d = Q.shape
    out = np.empty((U, G, n, d))
    lse = np.empty((U, G, n))
    S = np.zeros((U, n))
    for g in range(G):
        r = prefill(Q[:, g], K, V, scale, [alpha], M, R, nthreads=nthreads, lib=lib)
        out[:, g], lse[:, g] = r["out"], r["lse"]
        S += r["S"][:, 0]
    kept = np.stack([select(S[u], M, R, lib=lib) for u in range(U)])
    return {"out": out, "lse": lse, "S": S, "kept": kept}


class GroupCache(Cache):
    """The slot cache of ``Cache`` stepped by a group of query heads."""

    def step_group(self, q, k_new, v_new, alpha: float, force=None):
        """q [U, G, d]; k_new, v_new [U, d].  Steps (i)-(vi) of the generation step with G
        softmaxes over the same cached tokens; a token's score gains the sum of the G
        probabilities.  Returns out [U,G,d], info [U,3], scores [U,3] as ``Cache.step``."""
        q, k_new, v_new = _f64(q), _f64(k_new), _f64(v_new)
        U, G, d = q.shape
        out = np.empty((U, G, d))
        info = np.full((U, 3), -1, dtype=np.int32)
        sc3 = np.zeros((U, 3))
        for u in range(U):
            cnt, p = int(self.count[u]), int(self.len[u])
            Kall = np.vstack([self.K[u, :cnt], k_new[u:u + 1]])
            Vall = np.vstack([self.V[u, :cnt], v_new[u:u + 1]])
            gain = np.zeros(cnt + 1)
            for g in range(G):
                t = (Kall @ q[u, g]) * self.scale
                a = np.exp(t - t.max())
                a /= a.sum()
                out[u, g] = a @ Vall
                gain += a
            self.S[u, :cnt] = alpha * self.S[u, :cnt] + gain[:cnt]
            s_new = gain[cnt]
            if cnt < self.M:
                target = cnt
                self.count[u] = cnt + 1
            else:
                cand = [(self.S[u, s], int(self.pos[u, s]), s) for s in range(cnt)
                        if self.pos[u, s] <= p - self.R]
                if self.R == 0:
                    cand.append((s_new, p, -2))
                cand.sort(key=lambda c: (c[0], c[1]))
                info[u, 1], sc3[u, 1] = cand[0][2], cand[0][0]
                if len(cand) > 1:
                    info[u, 2], sc3[u, 2] = cand[1][2], cand[1][0]
                target = cand[0][2]
                if force is not None and force[u] != -3:
                    target = int(force[u])
                info[u, 0] = target
                sc3[u, 0] = s_new if target == -2 else self.S[u, target]
            if target >= 0:
                self.K[u, target], self.V[u, target] = k_new[u], v_new[u]
                self.S[u, target], self.pos[u, target] = s_new, p
            self.len[u] = p + 1
        return out, info, sc3
