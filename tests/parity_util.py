"""Lock-step comparison of the CUDA library with the fp64 oracle.

Both sides receive the same dtype-rounded inputs.  Index results must agree
exactly, except where the oracle's own competing scores are within 1e-5
relative of each other (a near-tie that fp32 cannot be asked to resolve); such a
step is counted as excused and the oracle is made to follow the library's choice
so that both continue from identical caches.

Tolerances: scores 1e-4 relative; attention output 2e-2 relative + 1e-3 absolute
for 16-bit storage, 1e-4 relative + 1e-5 absolute for fp32 storage.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

import oracle
from paper_2407_20485_b200 import binding as a2sf
from paper_2407_20485_b200 import workloads as wl

SCORE_RTOL = 1e-4
SCORE_ATOL = 1e-34
TIE_RTOL = 1e-5


def out_tolerance(dtype: str):
    return (1e-4, 1e-5) if dtype == "fp32" else (2e-2, 1e-3)


@dataclass
class ParityReport:
    units: int = 0
    steps: int = 0
    prefill_excused: int = 0
    decode_excused: int = 0
    decode_evictions: int = 0
    max_out_err: float = 0.0       # max |g-o| / (rtol*|o| + atol): must stay <= 1
    max_score_rel: float = 0.0
    notes: List[str] = field(default_factory=list)


def check_out(got: np.ndarray, want: np.ndarray, dtype: str, rep: ParityReport, what: str):
    rtol, atol = out_tolerance(dtype)
    err = np.abs(got - want) / (rtol * np.abs(want) + atol)
    worst = float(err.max()) if err.size else 0.0
    rep.max_out_err = max(rep.max_out_err, worst)
    assert worst <= 1.0, f"{what}: attention output off by {worst:.3g}x the tolerance"


def check_scores(got: np.ndarray, want: np.ndarray, rep: ParityReport, what: str):
    rel = np.abs(got - want) / (np.abs(want) + SCORE_ATOL / SCORE_RTOL)
    worst = float(rel.max()) if rel.size else 0.0
    rep.max_score_rel = max(rep.max_score_rel, worst)
    assert worst <= SCORE_RTOL, f"{what}: score relative error {worst:.3g} > {SCORE_RTOL}"


def check_kept(kept_g: np.ndarray, kept_o: np.ndarray, S_o: np.ndarray, n: int, M: int, R: int) -> int:
    """Kept sets of one unit.  Returns the number of excused swaps (0 = identical)."""
    assert kept_g.shape == kept_o.shape
    assert (np.diff(kept_g) > 0).all(), "kept_idx must be strictly ascending"
    assert kept_g.min() >= 0 and kept_g.max() < n
    if np.array_equal(kept_g, kept_o):
        return 0
    sg, so = set(kept_g.tolist()), set(kept_o.tolist())
    only_g, only_o = sorted(sg - so), sorted(so - sg)
    assert len(only_g) == len(only_o)
    cand_kept = [j for j in kept_o.tolist() if j < n - R]
    boundary = min(S_o[j] for j in cand_kept)
    for j in only_g + only_o:
        assert 0 <= j < n - R, f"recent / out-of-range token {j} differs"
        assert abs(S_o[j] - boundary) <= TIE_RTOL * abs(boundary), (
            f"kept sets differ at token {j}: oracle score {S_o[j]!r} vs boundary {boundary!r}")
    return len(only_g)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def make_inputs(w: wl.Workload, device, steps: int):
    """Prompt and decode tensors on ``device`` (generated there when large)."""
    gen_dev = device if w.units * w.n * w.d > (1 << 24) else "cpu"
    q, k, v = wl.make_prompt_chunked(w, gen_dev)
    q, k, v = q.to(device), k.to(device), v.to(device)
    if steps:
        dq, dk, dv = (t.to(device) for t in wl.make_decode(w, gen_dev, t_range=(0, steps)))
    else:
        dq = dk = dv = None
    return q, k, v, dq, dk, dv


def run_parity(w: wl.Workload, device="cuda", units: Optional[Sequence[int]] = None,
               alphas: Optional[Sequence[float]] = None, steps: Optional[int] = None,
               nthreads: Optional[int] = None, check_every: int = 1,
               inputs=None, alpha_units=None) -> ParityReport:
    """Prefill + cache build + ``steps`` decode steps on the GPU for ALL units of
    ``w``; the oracle follows the units listed in ``units`` (default: all).

    ``alphas``: extra forgetting factors whose scores / kept sets are checked through
    ``a2sf_rescore`` (the decode phase always uses ``w.alpha``).
    ``alpha_units``: float32 array [w.units], one forgetting factor per (batch, head): the
    per-head entry points are used and the oracle runs every unit with its own factor."""
    rep = ParityReport()
    nthreads = nthreads or oracle.host_threads()
    T = w.steps if steps is None else steps
    units = list(range(w.units)) if units is None else list(units)
    rep.units, rep.steps = len(units), T
    ub = [(u // w.H, u % w.H) for u in units]
    q, k, v, dq, dk, dv = inputs if inputs is not None else make_inputs(w, device, T)

    def pick(t):                      # [B,H,...] -> [len(units), ...] float64 on the host
        if len(units) == w.units:
            return to_f64(t).reshape((w.units,) + tuple(t.shape[2:]))
        return np.stack([to_f64(t[b, h]) for b, h in ub])

    def pick_i(t):
        a = t.detach().cpu().numpy().reshape((w.units,) + tuple(t.shape[2:]))
        return a[units]

    Qo, Ko, Vo = pick(q), pick(k), pick(v)

    # ---- prefill -------------------------------------------------------------------
    p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha)
    alphas_t = None
    if alpha_units is not None:
        alpha_units = np.asarray(alpha_units, dtype=np.float32)
        assert alpha_units.shape == (w.units,) and not alphas
        alphas_t = torch.from_numpy(alpha_units).view(w.B, w.H).to(device)
    out_g, S_g, kept_g, lse_g = a2sf.a2sf_prefill(p, q, k, v, alphas=alphas_t)
    torch.cuda.synchronize()
    all_alphas = [w.alpha] + [a for a in (alphas or []) if a != w.alpha]
    if alpha_units is None:
        ref = oracle.prefill(Qo, Ko, Vo, w.scale, all_alphas, w.budget, w.recent, sel_alpha=0,
                             nthreads=nthreads)
    else:
        per = [oracle.prefill(Qo[x:x + 1], Ko[x:x + 1], Vo[x:x + 1], w.scale, [float(alpha_units[uu])],
                              w.budget, w.recent) for x, uu in enumerate(units)]
        ref = {key: np.concatenate([r[key] for r in per]) for key in ("out", "lse", "S", "kept")}
        # the second pass alone, from the saved log-sum-exp, must give the same scores
        S2, kept2 = a2sf.a2sf_rescore(p, q, k, lse_g, alphas=alphas_t)
        torch.cuda.synchronize()
        assert torch.equal(S2, S_g) and torch.equal(kept2, kept_g)
    check_out(pick(out_g), ref["out"], w.dtype, rep, "prefill out")
    lse_err = np.abs(pick(lse_g) - ref["lse"]).max()
    assert lse_err <= 1e-4 * max(1.0, np.abs(ref["lse"]).max()), f"lse off by {lse_err}"
    check_scores(pick(S_g), ref["S"][:, 0], rep, f"prefill scores alpha={w.alpha}")
    kg = pick_i(kept_g)
    for x in range(len(units)):
        rep.prefill_excused += check_kept(kg[x], ref["kept"][x], ref["S"][x, 0], w.n, w.budget,
                                          w.recent)
    # forgetting-factor sweep through the second pass alone
    for ai, al in enumerate(all_alphas[1:], start=1):
        p2 = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, al)
        S2, kept2 = a2sf.a2sf_rescore(p2, q, k, lse_g)
        torch.cuda.synchronize()
        check_scores(pick(S2), ref["S"][:, ai], rep, f"rescore alpha={al}")
        k2 = pick_i(kept2)
        for x in range(len(units)):
            want = oracle.select(ref["S"][x, ai], w.budget, w.recent)
            rep.prefill_excused += check_kept(k2[x], want, ref["S"][x, ai], w.n, w.budget, w.recent)

    # ---- cache build: the oracle adopts the library's kept set (identical unless excused)
    cache = a2sf.Cache(p, device)
    cache.a2sf_cache_load(k, v, S_g, kept_g)
    ocache = oracle.Cache(len(units), w.d, w.budget, w.recent, w.scale)
    ocache.load(Ko, Vo, ref["S"][:, 0], kg)
    del Qo

    def compare_state(tag):
        st = cache.a2sf_cache_export()
        torch.cuda.synchronize()
        np.testing.assert_array_equal(pick_i(st["count"]), ocache.count, err_msg=f"{tag}: count")
        np.testing.assert_array_equal(pick_i(st["len"]), ocache.len, err_msg=f"{tag}: len")
        pos, S = pick_i(st["pos"]), pick(st["scores"])
        Kc, Vc = pick(st["k"]), pick(st["v"])
        for x in range(len(units)):
            c = int(ocache.count[x])
            np.testing.assert_array_equal(pos[x, :c], ocache.pos[x, :c],
                                          err_msg=f"{tag}: positions of unit {units[x]}")
            check_scores(S[x, :c], ocache.S[x, :c], rep, f"{tag}: cache scores")
            assert np.array_equal(Kc[x, :c], ocache.K[x, :c]), f"{tag}: K rows"
            assert np.array_equal(Vc[x, :c], ocache.V[x, :c]), f"{tag}: V rows"

    compare_state("after load")

    # ---- decode, lock-step ---------------------------------------------------------
    out_t = torch.empty((w.B, w.H, w.d), dtype=w.torch_dtype, device=device)
    ev_t = torch.empty((w.B, w.H), dtype=torch.int32, device=device)
    for t in range(T):
        if alphas_t is None:
            cache.a2sf_decode_step(w.alpha, dq[t], dk[t], dv[t], out_t, ev_t)
        else:
            cache.a2sf_decode_step_per_head(alphas_t, dq[t], dk[t], dv[t], out_t, ev_t)
        torch.cuda.synchronize()
        ev_g = pick_i(ev_t).astype(np.int32)
        force = np.where(ev_g == -1, -3, ev_g).astype(np.int32)
        step_alpha = w.alpha if alpha_units is None else [float(alpha_units[uu]) for uu in units]
        o_out, info, sc = ocache.step(pick(dq[t]), pick(dk[t]), pick(dv[t]), step_alpha, force=force,
                                      nthreads=nthreads)
        for x in range(len(units)):
            if info[x, 1] == -1:
                assert ev_g[x] == -1, f"step {t} unit {units[x]}: cache not full but evicted {ev_g[x]}"
                continue
            rep.decode_evictions += 1
            assert ev_g[x] != -1, f"step {t} unit {units[x]}: full cache but nothing evicted"
            if ev_g[x] != info[x, 1]:
                a_, b_ = sc[x, 0], sc[x, 1]
                assert abs(a_ - b_) <= TIE_RTOL * max(abs(a_), abs(b_)), (
                    f"step {t} unit {units[x]}: evicted slot {ev_g[x]} (score {a_!r}) but the "
                    f"rule picks {info[x, 1]} (score {b_!r})")
                rep.decode_excused += 1
        check_out(pick(out_t), o_out, w.dtype, rep, f"decode step {t} out")
        if (t + 1) % check_every == 0 or t == T - 1:
            compare_state(f"after step {t}")
    cache.close()
    return rep
