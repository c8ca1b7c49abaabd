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


# ---- the numpy parts of the oracle (streamed prompt, ideal similarity, grouped heads) ---------------
PY_SRC = Path(oracle.__file__).read_text()

PY_MUTANTS = {
    "ideal_keeps_the_smallest": ("order = np.lexsort((np.arange(m), -s_row))", "order = np.lexsort((np.arange(m), s_row))"),
    "ideal_tie_prefers_higher_position": ("order = np.lexsort((np.arange(m), -s_row))",
                                          "order = np.lexsort((-np.arange(m), -s_row))"),
    "ideal_row_not_normalised": ("    p[order] = w / w.sum()\n    return p", "    p[order] = w\n    return p"),
    "ideal_keeps_budget_not_budget_plus_one": ("ideal = ideal_row(s_row, M + 1)", "ideal = ideal_row(s_row, M)"),
    "policy_row_without_the_token_itself": ("seen = np.append(cache.pos[u, :cache.count[u]], i)",
                                            "seen = cache.pos[u, :cache.count[u]] if cache.count[u] else np.array([i])"),
    "cosine_without_norms": ("cos[u, i] = (meth @ ideal) / np.sqrt((meth @ meth) * (ideal @ ideal))",
                             "cos[u, i] = (meth @ ideal)"),
    "streamed_rows_use_the_previous_key": ("o, info[i], sc[i] = cache.step(Q[:, i], K[:, i], V[:, i], alpha,\n                                        force=None if force is None else force[i], nthreads=nthreads)\n        out[:, i] = o\n    return out, info, sc, cache",
                                           "o, info[i], sc[i] = cache.step(Q[:, i], K[:, max(i - 1, 0)], V[:, i], alpha,\n                                        force=None if force is None else force[i], nthreads=nthreads)\n        out[:, i] = o\n    return out, info, sc, cache"),
    "group_mean_instead_of_sum": ("                gain += a\n", "                gain += a / G\n"),
    "group_decay_after_add": ("self.S[u, :cnt] = alpha * self.S[u, :cnt] + gain[:cnt]",
                              "self.S[u, :cnt] = alpha * (self.S[u, :cnt] + gain[:cnt])"),
    "group_self_score_from_one_head": ("            s_new = gain[cnt]\n", "            s_new = a[cnt]\n"),
    "group_recent_window_off_by_one": ("if self.pos[u, s] <= p - self.R]", "if self.pos[u, s] < p - self.R]"),
    "group_prefill_keeps_one_head": ('        S += r["S"][:, 0]\n', '        S = r["S"][:, 0].copy()\n'),
}


def _py_pins(pins):
    pins.test_ideal_row_is_a_top_k_softmax()
    pins.test_similarity_is_one_while_nothing_is_pruned_and_bounded_after()
    pins.test_streamed_prompt_without_eviction_is_the_dense_prefill()
    pins.test_streamed_prompt_with_recent_equal_budget_is_a_sliding_window()
    pins.test_streamed_prompt_matches_a_mask_matrix_construction(6, 2, 0.5)
    pins.test_group_of_one_is_the_single_head_step()
    pins.test_group_scores_are_the_sum_of_the_heads_attention()
    pins.test_group_eviction_follows_the_summed_score()


def _load_py(tmp_path, name, src):
    import importlib.util

    real = Path(oracle.__file__).resolve().parent
    src = src.replace("_HERE = Path(__file__).resolve().parent", f"_HERE = Path({str(real)!r})")
    f = tmp_path / f"oracle_{name}.py"
    f.write_text(src)
    spec = importlib.util.spec_from_file_location(f"oracle_{name}", f)
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_unmodified_python_oracle_passes_its_pins(tmp_path, monkeypatch):
    import test_oracle_pins as pins

    monkeypatch.setattr(pins, "oracle", _load_py(tmp_path, "clean", PY_SRC))
    _py_pins(pins)


@pytest.mark.parametrize("name", sorted(PY_MUTANTS))
def test_python_oracle_mutant_is_caught(name, tmp_path, monkeypatch):
    import test_oracle_pins as pins

    old, new = PY_MUTANTS[name]
    assert PY_SRC.count(old) == 1, f"mutation site of {name} not found exactly once"
    monkeypatch.setattr(pins, "oracle", _load_py(tmp_path, name, PY_SRC.replace(old, new)))
    with pytest.raises(AssertionError):
        _py_pins(pins)
