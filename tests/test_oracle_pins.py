"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is an independent
statement (closed form, invariant, brute force from the materialised attention
matrix, or a library routine), not a re-typing of the oracle's own loops.
"""
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle

GOLDEN = Path(__file__).resolve().parent / "golden"


def _rand_unit(rng, n, d, heavy=True):
    Q = rng.standard_normal((n, d))
    K = rng.standard_normal((n, d))
    V = rng.standard_normal((n, d))
    if heavy:
        K[0] *= 4.0
        K[rng.integers(1, n)] *= 4.0
    return Q, K, V


def _brute_probs(Q, K, scale):
    """Causal softmax matrix written independently with numpy."""
    n = Q.shape[0]
    logits = (Q @ K.T) * scale
    P = np.zeros((n, n))
    for i in range(n):
        row = logits[i, : i + 1]
        e = np.exp(row - row.max())
        P[i, : i + 1] = e / e.sum()
    return P


def _brute_scores(P, alpha):
    """Eq. 5 term by term: A_{n,k} = sum_q alpha^(n-q) S_{q,k} (1-based q, k)."""
    n = P.shape[0]
    S = np.zeros(n)
    for k in range(1, n + 1):
        acc = 0.0
        for q in range(1, n + 1):
            w = 1.0 if n - q == 0 else alpha ** (n - q)
            acc += w * P[q - 1, k - 1]
        S[k - 1] = acc
    return S


# ---- p1: softmax rows sum to one; masked entries are zero (Eq. 3) ------------
def test_rows_sum_to_one_and_mask():
    rng = np.random.default_rng(1)
    Q, K, _ = _rand_unit(rng, 24, 16)
    P = oracle.attention_probs(Q, K, 0.25)
    assert np.abs(P.sum(axis=1) - 1.0).max() < 1e-12
    assert (np.triu(P, 1) == 0.0).all()
    assert (P >= 0).all()
    np.testing.assert_allclose(P, _brute_probs(Q, K, 0.25), rtol=1e-12, atol=1e-15)


# ---- p2: total score mass = sum of the weights (geometric series) -----------
@pytest.mark.parametrize("alpha", [0.0, 0.1, 0.5, 0.9, 1.0])
def test_score_mass_closed_form(alpha):
    rng = np.random.default_rng(2)
    n, d = 40, 8
    Q, K, V = _rand_unit(rng, n, d)
    _, _, S = oracle.prefill_rows(Q, K, V, 1 / np.sqrt(d), [alpha], 0, n)
    if alpha == 1.0:
        want = float(n)
    elif alpha == 0.0:
        want = 1.0
    else:
        want = (1 - alpha ** n) / (1 - alpha)
    assert abs(S[0].sum() - want) < 1e-11 * max(1.0, want)


# ---- p3 / p4 / p5: alpha = 1 -> column sums (H2O, Eq. 4); alpha = 0 -> last row;
#      general alpha -> Eq. 5 evaluated term by term from the materialised matrix
@pytest.mark.parametrize("n,d", [(5, 4), (16, 8), (13, 32)])
def test_brute_force_scores(n, d):
    rng = np.random.default_rng(100 + n)
    Q, K, V = _rand_unit(rng, n, d)
    scale = 1 / np.sqrt(d)
    P = _brute_probs(Q, K, scale)
    alphas = [1.0, 0.0, 0.3, 0.5, 0.9]
    out, lse, S = oracle.prefill_rows(Q, K, V, scale, alphas, 0, n)
    np.testing.assert_allclose(S[0], P.sum(axis=0), rtol=1e-12)            # Eq. 4
    np.testing.assert_allclose(S[1], P[n - 1], rtol=1e-12, atol=1e-300)   # alpha = 0
    for a, al in enumerate(alphas):
        np.testing.assert_allclose(S[a], _brute_scores(P, al), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(out, P @ V, rtol=1e-11, atol=1e-13)
    logits = (Q @ K.T) * scale
    for i in range(n):
        want = np.log(np.exp(logits[i, : i + 1]).sum())
        assert abs(lse[i] - want) < 1e-11 * max(1.0, abs(want))


# ---- p6 + golden: Q = 0 -> uniform rows -> exact rational scores -------------
def test_uniform_rows_golden():
    rows = [l.split() for l in (GOLDEN / "uniform_rows_scores.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    cases = {}
    for n, an, ad, j, sn, sd in rows:
        cases.setdefault((int(n), Fraction(int(an), int(ad))), {})[int(j)] = Fraction(int(sn), int(sd))
    assert len(cases) == 4
    rng = np.random.default_rng(3)
    for (n, alpha), want in cases.items():
        d = 8
        Q = np.zeros((n, d))
        K = rng.standard_normal((n, d))
        V = rng.standard_normal((n, d))
        out, lse, S = oracle.prefill_rows(Q, K, V, 0.3, [float(alpha)], 0, n)
        got = S[0]
        for j in range(n):
            assert abs(got[j] - float(want[j])) < 1e-14
        # uniform attention -> out_i is the running mean of V; lse_i = log(i+1)
        np.testing.assert_allclose(out, np.cumsum(V, 0) / np.arange(1, n + 1)[:, None], rtol=1e-12)
        np.testing.assert_allclose(lse, np.log(np.arange(1, n + 1)), atol=1e-14)


def test_harmonic_bias_alpha_one():
    # alpha = 1 and uniform rows: S_j = H_n - H_j, strictly decreasing in j -- the bias
    # towards early tokens that Sec. 3.1 describes.
    n, d = 32, 4
    Z = np.zeros((n, d))
    _, _, S = oracle.prefill_rows(Z, Z, Z, 1.0, [1.0], 0, n)
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, n + 1))])
    np.testing.assert_allclose(S[0], H[n] - H[:n], rtol=1e-13)
    assert (np.diff(S[0]) < 0).all()


# ---- p8: budget >= length -> dense causal attention (library routine) --------
def test_out_matches_sdpa_fp64():
    rng = np.random.default_rng(4)
    n, d = 48, 16
    Q, K, V = _rand_unit(rng, n, d)
    scale = 1 / np.sqrt(d)
    res = oracle.prefill(Q[None], K[None], V[None], scale, [0.5], M=n, R=4)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        is_causal=True, scale=scale)[0].numpy()
    np.testing.assert_allclose(res["out"][0], ref, rtol=1e-10, atol=1e-12)
    assert (res["kept"][0] == np.arange(n)).all()


def test_row_ranges_add_up():
    rng = np.random.default_rng(5)
    n, d = 30, 8
    Q, K, V = _rand_unit(rng, n, d)
    al = [0.5, 1.0]
    o_all, l_all, S_all = oracle.prefill_rows(Q, K, V, 0.4, al, 0, n)
    o_a, l_a, S_a = oracle.prefill_rows(Q, K, V, 0.4, al, 0, 11)
    o_b, l_b, S_b = oracle.prefill_rows(Q, K, V, 0.4, al, 11, n)
    np.testing.assert_allclose(S_a + S_b, S_all, rtol=1e-13)
    np.testing.assert_array_equal(np.concatenate([o_a, o_b]), o_all)
    np.testing.assert_array_equal(np.concatenate([l_a, l_b]), l_all)


# ---- p11: selection == sort on (S, position) --------------------------------
@pytest.mark.parametrize("n,M,R", [(50, 20, 10), (50, 20, 0), (50, 20, 20), (50, 1, 0), (50, 1, 1),
                                   (7, 20, 10), (20, 20, 5), (21, 20, 19)])
def test_selection_is_a_sort(n, M, R):
    rng = np.random.default_rng(n * 1000 + M * 10 + R)
    S = rng.random(n)
    S[rng.integers(0, n, 12)] = 0.25          # plenty of exact ties
    S[rng.integers(0, n, 6)] = 0.0
    kept = oracle.select(S, M, R)
    if n <= M:
        want = np.arange(n)
    else:
        cand = np.arange(n - R)
        order = cand[np.lexsort((cand, S[cand]))]          # primary S, secondary position
        want = np.sort(np.concatenate([order[n - M:], np.arange(n - R, n)]))
    np.testing.assert_array_equal(kept, want)
    assert len(kept) == min(n, M)
    assert (np.diff(kept) > 0).all()
    if n > M:
        assert set(range(n - R, n)) <= set(kept.tolist())


def test_selection_ties_drop_lowest_position_first():
    S = np.array([0.5, 0.1, 0.1, 0.1, 0.9, 0.1])
    # n=6, M=4, R=1: candidates 0..4, drop 2 smallest under (S, j): positions 1 and 2
    np.testing.assert_array_equal(oracle.select(S, 4, 1), [0, 3, 4, 5])


# ---- p7: prefill(n) + T decode steps == prefill(n+T) when nothing is evicted --
@pytest.mark.parametrize("alpha", [0.0, 0.3, 1.0])
def test_decode_recurrence_equals_eq5(alpha):
    rng = np.random.default_rng(6)
    n, T, d = 12, 9, 8
    Q, K, V = _rand_unit(rng, n + T, d)
    scale = 1 / np.sqrt(d)
    M = n + T
    full = oracle.prefill(Q[None], K[None], V[None], scale, [alpha], M=M, R=3)
    part = oracle.prefill(Q[None, :n], K[None, :n], V[None, :n], scale, [alpha], M=M, R=3)
    cache = oracle.Cache(1, d, M, 3, scale)
    cache.load(K[None, :n], V[None, :n], part["S"][:, 0], part["kept"])
    for t in range(T):
        out, info, _ = cache.step(Q[None, n + t], K[None, n + t], V[None, n + t], alpha)
        np.testing.assert_allclose(out[0], full["out"][0, n + t], rtol=1e-11, atol=1e-13)
        assert info[0, 0] == -1
    assert cache.count[0] == n + T and cache.len[0] == n + T
    np.testing.assert_array_equal(cache.pos[0], np.arange(n + T))
    np.testing.assert_allclose(cache.S[0], full["S"][0, 0], rtol=1e-11, atol=1e-300)


def test_decode_matches_brute_force_resum():
    """Decode simulated as 'append a row to the attention matrix and re-sum Eq. 5'."""
    rng = np.random.default_rng(7)
    n, T, d, alpha = 6, 5, 4, 0.6
    Q, K, V = _rand_unit(rng, n + T, d)
    scale = 0.5
    P = _brute_probs(Q, K, scale)
    M = n + T
    part = oracle.prefill(Q[None, :n], K[None, :n], V[None, :n], scale, [alpha], M=M, R=0)
    np.testing.assert_allclose(part["S"][0, 0], _brute_scores(P[:n, :n], alpha), rtol=1e-12)
    cache = oracle.Cache(1, d, M, 0, scale)
    cache.load(K[None, :n], V[None, :n], part["S"][:, 0], part["kept"])
    for t in range(T):
        cache.step(Q[None, n + t], K[None, n + t], V[None, n + t], alpha)
        m = n + t + 1
        np.testing.assert_allclose(cache.S[0, :m], _brute_scores(P[:m, :m], alpha), rtol=1e-12)


# ---- p9: recent == budget -> sliding-window attention ------------------------
def test_recent_equals_budget_is_sliding_window():
    rng = np.random.default_rng(8)
    n, T, d, W = 20, 25, 8, 6
    Q, K, V = _rand_unit(rng, n + T, d)
    scale = 1 / np.sqrt(d)
    pre = oracle.prefill(Q[None, :n], K[None, :n], V[None, :n], scale, [0.5], M=W, R=W)
    np.testing.assert_array_equal(pre["kept"][0], np.arange(n - W, n))
    cache = oracle.Cache(1, d, W, W, scale)
    cache.load(K[None, :n], V[None, :n], pre["S"][:, 0], pre["kept"])
    for t in range(T):
        p = n + t
        out, info, _ = cache.step(Q[None, p], K[None, p], V[None, p], 0.5)
        lo = p - W                                  # window: W cached tokens + the new one
        logits = (K[lo: p + 1] @ Q[p]) * scale
        a = np.exp(logits - logits.max())
        a /= a.sum()
        np.testing.assert_allclose(out[0], a @ V[lo: p + 1], rtol=1e-11, atol=1e-13)
        assert sorted(cache.pos[0].tolist()) == list(range(p - W + 1, p + 1))


# ---- p10: policy invariants under eviction -----------------------------------
@pytest.mark.parametrize("M,R", [(8, 4), (8, 0), (8, 8), (8, 1), (1, 0), (1, 1), (5, 2)])
def test_decode_invariants(M, R):
    rng = np.random.default_rng(9 + M * 10 + R)
    n, T, d, alpha = 14, 30, 8, 0.5
    U = 3
    Q = rng.standard_normal((U, n + T, d))
    K = rng.standard_normal((U, n + T, d))
    V = rng.standard_normal((U, n + T, d))
    K[:, 0] *= 4
    scale = 1 / np.sqrt(d)
    pre = oracle.prefill(Q[:, :n], K[:, :n], V[:, :n], scale, [alpha], M=M, R=R, nthreads=2)
    cache = oracle.Cache(U, d, M, R, scale)
    cache.load(K[:, :n], V[:, :n], pre["S"][:, 0], pre["kept"])
    for t in range(T):
        p = n + t
        before = cache.snapshot()
        out, info, sc = cache.step(Q[:, p], K[:, p], V[:, p], alpha, nthreads=2)
        for u in range(U):
            assert cache.len[u] == p + 1
            assert cache.count[u] == min(p + 1, M)
            pos = cache.pos[u, : cache.count[u]]
            assert len(set(pos.tolist())) == len(pos)
            # the R newest positions are resident
            assert set(range(p - R + 1, p + 1)) <= set(pos.tolist())
            assert (cache.S[u, : cache.count[u]] >= 0).all()
            ev = info[u, 0]
            assert ev == info[u, 1]
            if ev >= 0:
                old_pos = before["pos"][u, ev]
                assert old_pos <= p - R                           # never evict a recent token
                assert cache.pos[u, ev] == p
                # the evicted one is the (S, pos) minimum of the candidates: rebuild the
                # post-update scores (the vacated slot's score is reported separately)
                post = cache.S[u].copy()
                post[ev] = sc[u, 0]
                cand = [s for s in range(M) if before["pos"][u, s] <= p - R]
                keys = [(post[s], before["pos"][u, s]) for s in cand]
                if R == 0:
                    cand.append(-2)
                    keys.append((cache.S[u, ev], p))
                assert cand[min(range(len(cand)), key=lambda t: keys[t])] == ev
            elif ev == -2:
                assert R == 0
                np.testing.assert_array_equal(cache.pos[u], before["pos"][u])


def test_step_probabilities_sum_to_one_and_alpha0_keeps_latest_row():
    rng = np.random.default_rng(10)
    d, M = 8, 16
    Kc = rng.standard_normal((1, 10, d))
    Vc = rng.standard_normal((1, 10, d))
    cache = oracle.Cache(1, d, M, 2, 0.3)
    cache.load(Kc, Vc, rng.random((1, 10)), np.arange(10, dtype=np.int32)[None])
    S0 = cache.S.copy()
    q, k, v = rng.standard_normal((3, 1, d))
    cache.step(q, k, v, 0.7)
    a = cache.S[0, :11] - np.concatenate([0.7 * S0[0, :10], [0.0]])
    assert abs(a.sum() - 1.0) < 1e-12
    logits = np.concatenate([Kc[0] @ q[0], k @ q[0]]) * 0.3
    want = np.exp(logits - logits.max())
    want /= want.sum()
    np.testing.assert_allclose(a, want, rtol=1e-10)
    # alpha = 0: the score is exactly the latest attention row (Sec. 4.4.2)
    q2, k2, v2 = rng.standard_normal((3, 1, d))
    cache.step(q2, k2, v2, 0.0)
    logits = np.concatenate([cache.K[0, :12] @ q2[0]]) * 0.3
    want = np.exp(logits - logits.max())
    want /= want.sum()
    np.testing.assert_allclose(cache.S[0, :12], want, rtol=1e-12)


def test_slot_permutation_invariance():
    rng = np.random.default_rng(11)
    d, M, R, n = 8, 10, 3, 10
    K = rng.standard_normal((1, n, d))
    V = rng.standard_normal((1, n, d))
    S = rng.random((1, n))
    perm = rng.permutation(n).astype(np.int32)
    a = oracle.Cache(1, d, M, R, 0.35)
    b = oracle.Cache(1, d, M, R, 0.35)
    a.load(K, V, S, np.arange(n, dtype=np.int32)[None])
    b.load(K, V, S, perm[None])
    for t in range(12):
        q, k, v = rng.standard_normal((3, 1, d))
        pa = a.pos.copy()
        pb = b.pos.copy()
        oa, ia, _ = a.step(q, k, v, 0.5)
        ob, ib, _ = b.step(q, k, v, 0.5)
        np.testing.assert_allclose(oa, ob, rtol=1e-12, atol=1e-14)
        assert pa[0, ia[0, 0]] == pb[0, ib[0, 0]]            # same evicted POSITION
        sa = dict(zip(a.pos[0].tolist(), a.S[0].tolist()))
        sb = dict(zip(b.pos[0].tolist(), b.S[0].tolist()))
        assert sa.keys() == sb.keys()
        for k_ in sa:
            assert abs(sa[k_] - sb[k_]) <= 1e-13 * max(1.0, abs(sa[k_]))


def test_new_token_can_be_dropped_only_when_recent_is_zero():
    d, M = 4, 3
    cache = oracle.Cache(1, d, M, 0, 1.0)
    K = np.eye(3, d)[None] * 5.0
    cache.load(K, np.ones((1, 3, d)), np.array([[5.0, 6.0, 7.0]]), np.arange(3, dtype=np.int32)[None])
    q = np.array([[1.0, 1.0, 1.0, 0.0]])
    k_new = np.array([[-9.0, -9.0, -9.0, 0.0]])              # negligible self-attention
    out, info, sc = cache.step(q, k_new, np.zeros((1, d)), 1.0)
    assert info[0, 0] == -2 and cache.count[0] == 3 and cache.len[0] == 4
    np.testing.assert_array_equal(cache.pos[0], [0, 1, 2])


def test_forced_eviction_reports_rule_choice():
    rng = np.random.default_rng(12)
    d, M, R = 4, 4, 1
    cache = oracle.Cache(1, d, M, R, 0.5)
    cache.load(rng.standard_normal((1, 4, d)), rng.standard_normal((1, 4, d)),
               np.array([[0.4, 0.1, 0.3, 0.2]]), np.arange(4, dtype=np.int32)[None])
    snap = cache.snapshot()
    q, k, v = rng.standard_normal((3, 1, d))
    _, info, _ = cache.step(q, k, v, 0.5)
    rule = info[0, 0]
    cache.restore(snap)
    other = (rule + 1) % 3
    _, info2, sc2 = cache.step(q, k, v, 0.5, force=np.array([other], dtype=np.int32))
    assert info2[0, 0] == other and info2[0, 1] == rule
    assert cache.pos[0, other] == 4 and cache.pos[0, rule] == snap["pos"][0, rule]
    assert sc2[0, 1] <= sc2[0, 0]


def test_batch_threads_do_not_change_results():
    rng = np.random.default_rng(13)
    U, n, d = 5, 20, 8
    Q, K, V = rng.standard_normal((3, U, n, d))
    a = oracle.prefill(Q, K, V, 0.3, [0.5, 1.0], M=8, R=4, sel_alpha=1, nthreads=1)
    b = oracle.prefill(Q, K, V, 0.3, [0.5, 1.0], M=8, R=4, sel_alpha=1, nthreads=4)
    for key in ("out", "lse", "S", "kept"):
        np.testing.assert_array_equal(a[key], b[key])
    for u in range(U):
        np.testing.assert_array_equal(a["kept"][u], oracle.select(a["S"][u, 1], 8, 4))


def test_per_unit_alpha_equals_unit_by_unit_scalar_steps():
    """A vector of forgetting factors is the scalar step applied unit by unit."""
    rng = np.random.default_rng(14)
    U, d, M, R = 3, 8, 6, 2
    K, V = rng.standard_normal((2, U, M, d))
    S = rng.random((U, M))
    kept = np.tile(np.arange(M, dtype=np.int32), (U, 1))
    alphas = [0.0, 0.4, 1.0]
    a = oracle.Cache(U, d, M, R, 0.3)
    a.load(K, V, S, kept)
    singles = []
    for u in range(U):
        c = oracle.Cache(1, d, M, R, 0.3)
        c.load(K[u:u + 1], V[u:u + 1], S[u:u + 1], kept[u:u + 1])
        singles.append(c)
    for t in range(5):
        q, k, v = rng.standard_normal((3, U, d))
        out, info, sc = a.step(q, k, v, alphas)
        for u in range(U):
            o1, i1, s1 = singles[u].step(q[u:u + 1], k[u:u + 1], v[u:u + 1], alphas[u])
            np.testing.assert_array_equal(out[u], o1[0])
            np.testing.assert_array_equal(info[u], i1[0])
            np.testing.assert_array_equal(a.S[u], singles[u].S[0])
            np.testing.assert_array_equal(a.pos[u], singles[u].pos[0])


# ---- prompt pruned row by row (streamed prefill) ------------------------------------------------
def test_streamed_prompt_without_eviction_is_the_dense_prefill():
    """While the budget holds the whole prompt nothing is evicted, so processing it token by
    token must reproduce dense causal attention (Eq. 3) and the scores of Eq. 5."""
    rng = np.random.default_rng(21)
    n, d, alpha = 23, 8, 0.7
    Q, K, V = _rand_unit(rng, n, d)
    out, info, _, cache = oracle.streaming_prefill(Q[None], K[None], V[None], 0.35, alpha, M=n, R=5)
    P = _brute_probs(Q, K, 0.35)
    np.testing.assert_allclose(out[0], P @ V, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(cache.S[0], _brute_scores(P, alpha), rtol=1e-12, atol=1e-15)
    np.testing.assert_array_equal(cache.pos[0], np.arange(n))
    assert (info[:, 0, 0] == -1).all() and cache.count[0] == n and cache.len[0] == n


def test_streamed_prompt_with_recent_equal_budget_is_a_sliding_window():
    """R = M: every step drops the oldest token, so row i sees tokens i-M .. i only."""
    rng = np.random.default_rng(22)
    n, d, M = 30, 4, 6
    Q, K, V = _rand_unit(rng, n, d)
    out, _, _, _ = oracle.streaming_prefill(Q[None], K[None], V[None], 0.5, 0.4, M=M, R=M)
    for i in range(n):
        lo = max(0, i - M)
        s = (K[lo:i + 1] @ Q[i]) * 0.5
        w = np.exp(s - s.max())
        np.testing.assert_allclose(out[0, i], (w / w.sum()) @ V[lo:i + 1], rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("M,R,alpha", [(6, 2, 0.5), (5, 0, 0.8), (7, 3, 1.0), (4, 1, 0.0)])
def test_streamed_prompt_matches_a_mask_matrix_construction(M, R, alpha):
    """The same policy written the way the paper draws it: an n x n mask built row by row over
    full-length score vectors (no slots, no cache object)."""
    rng = np.random.default_rng(23 + M)
    n, d, scale = 26, 6, 0.4
    Q, K, V = _rand_unit(rng, n, d)
    out, info, _, cache = oracle.streaming_prefill(Q[None], K[None], V[None], scale, alpha, M=M, R=R)
    alive = np.zeros(n, dtype=bool)
    S = np.zeros(n)
    for i in range(n):
        alive[i] = True
        idx = np.flatnonzero(alive)
        s = (K[idx] @ Q[i]) * scale
        w = np.exp(s - s.max())
        w /= w.sum()
        np.testing.assert_allclose(out[0, i], w @ V[idx], rtol=1e-11, atol=1e-12)
        S *= alpha
        S[idx] += w
        if alive.sum() > M:
            cand = [j for j in idx if j <= i - R]              # outside the recent window
            victim = min(cand, key=lambda j: (S[j], j))
            alive[victim] = False
            S[victim] = 0.0
    kept = np.sort(cache.pos[0, :cache.count[0]])
    np.testing.assert_array_equal(kept, np.flatnonzero(alive))
    order = np.argsort(cache.pos[0, :cache.count[0]])
    np.testing.assert_allclose(cache.S[0, :cache.count[0]][order], S[alive], rtol=1e-11, atol=1e-14)


def test_streamed_prompt_differs_from_one_shot_selection():
    """With a budget below the prompt length the two readings part: a token evicted early cannot
    be attended to later, so outputs of late rows differ from dense attention."""
    rng = np.random.default_rng(29)
    n, d = 40, 8
    Q, K, V = _rand_unit(rng, n, d)
    out, _, _, _ = oracle.streaming_prefill(Q[None], K[None], V[None], 0.35, 0.5, M=8, R=4)
    dense = _brute_probs(Q, K, 0.35) @ V
    np.testing.assert_allclose(out[0, :9], dense[:9], rtol=1e-12, atol=1e-13)   # nothing evicted yet
    assert np.abs(out[0, 20:] - dense[20:]).max() > 1e-3


# ---- similarity with the ideal mask (Sec. 4.3) --------------------------------------------------
def test_ideal_row_is_a_top_k_softmax():
    rng = np.random.default_rng(31)
    s = rng.standard_normal(40)
    s[7] = s[3]                                             # a tie: the lower position is kept first
    for keep in (1, 5, 39, 40, 100):
        p = oracle.ideal_row(s, keep)
        k = min(keep, 40)
        assert np.count_nonzero(p) == k and abs(p.sum() - 1) < 1e-14
        kept = np.flatnonzero(p)
        assert s[kept].min() >= np.delete(s, kept).max(initial=-np.inf)
        t = torch.softmax(torch.from_numpy(s[kept]), 0).numpy()
        np.testing.assert_allclose(p[kept], t, rtol=1e-13)
    sel = np.zeros(40); sel[[3, 7]] = 1
    s2 = np.where(sel > 0, 5.0, s - 10)                     # positions 3 and 7 tie at the top
    assert np.flatnonzero(oracle.ideal_row(s2, 1)).tolist() == [3]


def test_similarity_is_one_while_nothing_is_pruned_and_bounded_after():
    rng = np.random.default_rng(32)
    n, d, M = 30, 8, 10
    Q, K, V = _rand_unit(rng, n, d)
    cos, out, _, _, _ = oracle.ideal_similarity(Q[None], K[None], V[None], 0.35, 0.5, M=M, R=5)
    np.testing.assert_allclose(cos[0, :M + 1], 1.0, rtol=0, atol=1e-14)   # rows that see every token
    assert (cos > 0).all() and (cos <= 1 + 1e-14).all()
    ref, _, _, _ = oracle.streaming_prefill(Q[None], K[None], V[None], 0.35, 0.5, M=M, R=5)
    np.testing.assert_array_equal(out, ref)                                # the diagnostic changes nothing
    full, *_ = oracle.ideal_similarity(Q[None], K[None], V[None], 0.35, 0.5, M=n, R=5)
    np.testing.assert_allclose(full, 1.0, rtol=0, atol=1e-14)


def test_similarity_orders_the_policies_on_a_sink_plus_recency_pattern():
    """A prompt whose rows attend to token 0 (a sink), to two tokens that matter for a while and
    to their neighbourhood: the sliding window loses the sink, pure accumulation (alpha = 1)
    clings to early tokens, the forgetting factor follows the ideal mask most closely."""
    rng = np.random.default_rng(33)
    n, d, M = 96, 16, 12
    K = rng.standard_normal((n, d))
    Q = rng.standard_normal((n, d))
    K[0] *= 0.2
    e = np.zeros(d); e[0] = 6.0
    K[0] += e; Q[:, 0] = 1.0                                   # every row likes token 0
    for i in range(n):                                         # rows like a token some 20 rows back ...
        j = max(0, i - 20 - (i % 7))
        Q[i] += 0.9 * K[j]
        if i >= 2:
            Q[i] += 0.5 * K[i - 1]                             # ... and their predecessor
    V = rng.standard_normal((n, d))
    res = {}
    for name, (alpha, R) in {"local": (1.0, M), "h2o": (1.0, M // 2), "a2sf": (0.6, 0)}.items():
        cos, *_ = oracle.ideal_similarity(Q[None], K[None], V[None], 0.25, alpha, M=M, R=R)
        res[name] = cos[0, M + 1:].mean()
    assert res["local"] < res["h2o"] < res["a2sf"], res


# ---- grouped query heads ------------------------------------------------------------------------
def test_group_of_one_is_the_single_head_step():
    rng = np.random.default_rng(41)
    U, d, M, R = 3, 8, 6, 2
    K, V = rng.standard_normal((2, U, M, d))
    S = rng.random((U, M))
    kept = np.tile(np.arange(M, dtype=np.int32), (U, 1))
    a, b = oracle.Cache(U, d, M, R, 0.3), oracle.GroupCache(U, d, M, R, 0.3)
    a.load(K, V, S, kept); b.load(K, V, S, kept)
    for t in range(8):
        q, k, v = rng.standard_normal((3, U, d))
        o1, i1, s1 = a.step(q, k, v, 0.6)
        o2, i2, s2 = b.step_group(q[:, None], k, v, 0.6)
        np.testing.assert_allclose(o2[:, 0], o1, rtol=1e-13, atol=1e-15)
        np.testing.assert_array_equal(i2, i1)
        np.testing.assert_allclose(s2, s1, rtol=1e-13)
        np.testing.assert_allclose(b.S, a.S, rtol=1e-13)
        np.testing.assert_array_equal(b.pos, a.pos)


def test_group_scores_are_the_sum_of_the_heads_attention():
    """Prefill: S = sum_g of Eq. 5 per head, from independently built attention matrices.
    Decode without eviction: prefill(n) + T grouped steps == prefill(n + T)."""
    rng = np.random.default_rng(42)
    G, n, T, d, alpha, scale = 3, 14, 6, 8, 0.7, 0.3
    Q = rng.standard_normal((G, n + T, d))
    K, V = rng.standard_normal((2, n + T, d))
    K[0] *= 3
    full = oracle.group_prefill(Q[None], K[None], V[None], scale, alpha, M=64, R=4)
    want = sum(_brute_scores(_brute_probs(Q[g], K, scale), alpha) for g in range(G))
    np.testing.assert_allclose(full["S"][0], want, rtol=1e-12)
    for g in range(G):
        np.testing.assert_allclose(full["out"][0, g], _brute_probs(Q[g], K, scale) @ V, rtol=1e-12, atol=1e-14)
    head = oracle.group_prefill(Q[None, :, :n], K[None, :n], V[None, :n], scale, alpha, M=64, R=4)
    c = oracle.GroupCache(1, d, 64, 4, scale)
    c.load(K[None, :n], V[None, :n], head["S"], head["kept"])
    for t in range(n, n + T):
        o, info, _ = c.step_group(Q[None, :, t], K[None, t], V[None, t], alpha)
        np.testing.assert_allclose(o[0], full["out"][0, :, t], rtol=1e-12, atol=1e-14)
        assert info[0, 0] == -1
    np.testing.assert_allclose(c.S[0, :n + T], full["S"][0], rtol=1e-12)


def test_group_eviction_follows_the_summed_score():
    """Two heads that each favour a different old token keep both; the token neither looks at goes."""
    d, M = 4, 3
    e = np.eye(d)
    K = np.stack([e[0], e[1], e[2]]) * 4.0
    c = oracle.GroupCache(1, d, M, 1, 1.0)
    c.load(K[None], K[None], np.full((1, 3), 0.5), np.arange(3, dtype=np.int32)[None])
    q = np.stack([e[0], e[1]]) * 4.0                       # head 0 -> token 0, head 1 -> token 1
    out, info, sc = c.step_group(q[None], (e[3] * 4.0)[None], e[3][None], 0.5)
    assert info[0, 0] == 2                                  # token 2 had the lowest summed score
    assert sorted(c.pos[0].tolist()) == [0, 1, 3]
    # the same step with a single head (head 0 only) would have dropped token 1 or 2, lowest position first
    c1 = oracle.GroupCache(1, d, M, 1, 1.0)
    c1.load(K[None], K[None], np.full((1, 3), 0.5), np.arange(3, dtype=np.int32)[None])
    _, info1, _ = c1.step_group(q[None, :1], (e[3] * 4.0)[None], e[3][None], 0.5)
    assert info1[0, 0] == 1
