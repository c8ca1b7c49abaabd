"""The pins bite: plausible mistakes planted in a COPY of the oracle are caught.

Each mutant is the oracle source with one line changed (a dropped term, a wrong sign or
index, a swapped order).  It is compiled on the CPU into its own library and run through a
compact set of the pins; every mutant must fail at least one of them, and the unmodified
source must pass all of them.  Nothing here touches the CUDA library.
"""
from pathlib import Path

import numpy as np
import pytest

import oracle

SRC = (Path(oracle.__file__).resolve().parent / "a2sf_oracle.c").read_text()

MUTANTS = {
    "weight_exponent_off_by_one": ("wa[n - 1] = 1.0;", "wa[n - 1] = alphas[a];"),
    "diagonal_term_dropped": ("for (int j = 0; j <= i; ++j) Sa[j] += wi * P[j];",
                              "for (int j = 0; j < i; ++j) Sa[j] += wi * P[j];"),
    "scale_dropped": ("        s *= scale;\n        P[j] = s;", "        P[j] = s;"),
    "key_index_wrong": ("const double *k = K + (size_t)j * d;\n        double s = 0.0;",
                        "const double *k = K + (size_t)i * d;\n        double s = 0.0;"),
    "rows_not_normalised": ("    for (int j = 0; j <= i; ++j) P[j] /= l;\n    return m + log(l);",
                            "    return m + log(l);"),
    "lse_without_max": ("    return m + log(l);", "    return log(l);"),
    "tie_break_reversed": ("    return (x->j > y->j) - (x->j < y->j);", "    return (x->j < y->j) - (x->j > y->j);"),
    "drops_one_too_many": ("    int drop = n - M;", "    int drop = n - M + 1;"),
    "largest_dropped_instead_of_smallest": ("for (int r = drop; r < ncand; ++r) kept[m++] = c[r].j;",
                                            "for (int r = 0; r < ncand - drop; ++r) kept[m++] = c[r].j;"),
    "decay_after_add": ("Sc[s] = alpha * Sc[s] + a[s];", "Sc[s] = alpha * (Sc[s] + a[s]);"),
    "recent_window_off_by_one": ("if (t < cnt && !(ps <= p - R)) continue;", "if (t < cnt && !(ps < p - R)) continue;"),
    "self_score_dropped": ("    double s_new = a[cnt];", "    double s_new = 0.0;"),
    "self_logit_missing_from_softmax": ("    for (int s = 0; s <= cnt; ++s) { a[s] = exp(a[s] - m); l += a[s]; }",
                                        "    for (int s = 0; s <= cnt; ++s) { a[s] = exp(a[s] - m); if (s < cnt) l += a[s]; }"),
    "decode_tie_break_by_slot_not_position": ("int lt_best = (best == -1) || sc < bs || (sc == bs && ps < bp);",
                                              "int lt_best = (best == -1) || sc < bs;"),
    "new_token_written_before_length_read": ("        pos[target] = p;", "        pos[target] = p + 1;"),
}


def _build(tmp_path, name, src):
    c = tmp_path / f"{name}.c"
    so = tmp_path / f"lib_{name}.so"
    c.write_text(src)
    import subprocess

    subprocess.run(["gcc", "-O2", "-fPIC", "-shared", "-std=c11", "-pthread", str(c), "-o", str(so), "-lm"],
                   check=True)
    return oracle.load(so)


def _probs(Q, K, scale):
    n = Q.shape[0]
    L = (Q @ K.T) * scale
    P = np.zeros((n, n))
    for i in range(n):
        e = np.exp(L[i, : i + 1] - L[i, : i + 1].max())
        P[i, : i + 1] = e / e.sum()
    return P


def _scores(P, alpha):
    n = P.shape[0]
    w = np.array([1.0 if i == n - 1 else alpha ** (n - 1 - i) for i in range(n)])
    return (w[:, None] * P).sum(0)


def run_pins(lib):
    """A compact version of the pins; raises AssertionError on the first violation."""
    rng = np.random.default_rng(7)
    n, d = 14, 8
    Q, K, V = rng.standard_normal((3, n, d))
    K[0] *= 4
    scale = 0.4
    P = _probs(Q, K, scale)
    # materialised rows, closed-form mass, Eq. 5 by brute force, output, lse
    Po = oracle.attention_probs(Q, K, scale, lib=lib)
    assert np.abs(Po.sum(1) - 1).max() < 1e-12
    np.testing.assert_allclose(Po, P, rtol=1e-11, atol=1e-14)
    alphas = [1.0, 0.0, 0.3]
    out, lse, S = oracle.prefill_rows(Q, K, V, scale, alphas, 0, n, lib=lib)
    for a, al in enumerate(alphas):
        np.testing.assert_allclose(S[a], _scores(P, al), rtol=1e-11, atol=1e-300)
    np.testing.assert_allclose(out, P @ V, rtol=1e-10, atol=1e-13)
    L = (Q @ K.T) * scale
    np.testing.assert_allclose(lse, [np.log(np.exp(L[i, : i + 1]).sum()) for i in range(n)], rtol=1e-11)
    # selection == sort on (score, position), with exact ties
    Ssel = np.array([0.5, 0.1, 0.1, 0.1, 0.9, 0.1, 0.3, 0.2])
    np.testing.assert_array_equal(oracle.select(Ssel, 5, 2, lib=lib), [0, 4, 5, 6, 7])
    # prefill(n0) + decode steps == prefill(n) when nothing is evicted
    n0 = 9
    for alpha in (0.0, 0.6, 1.0):
        full = oracle.prefill(Q[None], K[None], V[None], scale, [alpha], M=n, R=3, lib=lib)
        part = oracle.prefill(Q[None, :n0], K[None, :n0], V[None, :n0], scale, [alpha], M=n, R=3, lib=lib)
        cache = oracle.Cache(1, d, n, 3, scale, lib=lib)
        cache.load(K[None, :n0], V[None, :n0], part["S"][:, 0], part["kept"])
        for t in range(n0, n):
            o, info, _ = cache.step(Q[None, t], K[None, t], V[None, t], alpha)
            np.testing.assert_allclose(o[0], full["out"][0, t], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(cache.S[0], full["S"][0, 0], rtol=1e-10, atol=1e-300)
        np.testing.assert_array_equal(cache.pos[0], np.arange(n))
    # recent == budget: the cache is the sliding window of the W newest tokens
    W = 4
    pre = oracle.prefill(Q[None, :n0], K[None, :n0], V[None, :n0], scale, [0.5], M=W, R=W, lib=lib)
    cache = oracle.Cache(1, d, W, W, scale, lib=lib)
    cache.load(K[None, :n0], V[None, :n0], pre["S"][:, 0], pre["kept"])
    for t in range(n0, n):
        cache.step(Q[None, t], K[None, t], V[None, t], 0.5)
        assert sorted(cache.pos[0].tolist()) == list(range(t - W + 1, t + 1))
    # eviction picks the (score, position) minimum of the non-recent slots: equal scores -> lowest position
    cache = oracle.Cache(1, d, 4, 1, 1.0, lib=lib)
    Kc = np.zeros((1, 4, d))
    cache.load(Kc, np.ones((1, 4, d)), np.array([[0.5, 0.2, 0.2, 0.9]]), np.array([[3, 2, 1, 0]], dtype=np.int32))
    cache.len[0] = 4
    _, info, _ = cache.step(np.zeros((1, d)), np.zeros((1, d)), np.zeros((1, d)), 1.0)
    assert info[0, 0] == 2           # slots 1 and 2 tie on the score; slot 2 holds the lower position
    assert cache.pos[0, 2] == 4 and abs(cache.S[0, 2] - 0.2) < 1e-12      # new token: a_self = 1/5


def test_unmodified_oracle_passes_the_compact_pins(tmp_path):
    run_pins(_build(tmp_path, "clean", SRC))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(tmp_path, name):
    old, new = MUTANTS[name]
    assert SRC.count(old) >= 1, f"mutation site of {name} not found in the oracle source"
    lib = _build(tmp_path, name, SRC.replace(old, new, 1))
    with pytest.raises(AssertionError):
        run_pins(lib)
