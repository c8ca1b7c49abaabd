"""The allocation-free prefill entry point against the oracle and the regular entry point.

Collected last on purpose (file name), so a run that stops at the first failure has
already exercised everything else.  Callers such as an inference engine whose own
pool allocator owns the GPU cannot call cudaMalloc; for them the library keeps the
prefill's log-sum-exp scratch in a fixed array of its device image.  The test calls
the entry point twice in a row with different shapes -- the second call finds the
first call's leftovers in the shared array -- and both times demands the oracle's
results (and, within the same tolerances, the regular entry point's).
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(a2sf, wl, w, **params):
    import oracle
    from parity_util import ParityReport, check_kept, check_out, check_scores, to_f64

    q, k, v = (t.cuda() for t in wl.make_prompt(w))
    p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha, **params)
    ref_out, ref_S, ref_kept, _ = a2sf.a2sf_prefill(p, q, k, v)
    # the caller owns every buffer: allocate them before the call under test
    out = torch.empty_like(q)
    S = torch.empty_like(ref_S)
    kept = torch.empty_like(ref_kept)
    torch.cuda.synchronize()
    # The driver's own count of free device memory sees every allocation, whoever makes it
    # (torch's counters would only see torch's).  The first call on a device looks up the
    # array's address, so the comparison is taken around a second, identical call.
    rc = a2sf.a2sf_prefill_static_scratch(p, q, k, v, out, S, kept)
    torch.cuda.synchronize()
    assert rc == a2sf.A2SF_OK, a2sf.status_string(rc)
    free_before, _ = torch.cuda.mem_get_info()
    rc = a2sf.a2sf_prefill_static_scratch(p, q, k, v, out, S, kept)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert rc == a2sf.A2SF_OK, a2sf.status_string(rc)
    assert free_after == free_before, "the call changed the amount of free device memory"
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK

    # against the oracle, at the tolerances of every other parity test
    U, n = w.units, w.n
    Q, K, V = (to_f64(t).reshape(U, n, w.d) for t in (q, k, v))
    i0 = max(0, n - p.score_window) if p.score_window > 0 else 0
    rep = ParityReport()
    if i0 == 0:
        ref = oracle.prefill(Q, K, V, w.scale, [w.alpha], w.budget, w.recent, nthreads=oracle.host_threads())
        want_out, want_S, want_kept = ref["out"], ref["S"][:, 0], ref["kept"]
    else:       # truncated scoring window: the partial sum over the last rows, selection on it
        rows = [oracle.prefill_rows(Q[u], K[u], V[u], w.scale, [w.alpha], 0, n) for u in range(U)]
        want_out = np.stack([r[0] for r in rows])
        want_S = np.stack([oracle.prefill_rows(Q[u], K[u], V[u], w.scale, [w.alpha], i0, n)[2][0] for u in range(U)])
        want_kept = np.stack([oracle.select(want_S[u], w.budget, w.recent) for u in range(U)])
    check_out(to_f64(out).reshape(U, n, w.d), want_out, w.dtype, rep, "static-scratch out")
    check_scores(to_f64(S).reshape(U, n), want_S, rep, "static-scratch scores")
    kg = kept.cpu().numpy().reshape(U, -1)
    for u in range(U):
        check_kept(kg[u], want_kept[u], want_S[u], n, w.budget, w.recent)
    # and against the regular entry point.  For bf16 storage with d = 128 the two run different
    # forms of the P V product (no workspace here, hence no fp16 copy of V: two bf16 terms), so
    # outputs agree within the tolerance, not bit for bit; the scoring pass is the same kernel.
    torch.testing.assert_close(S, ref_S, rtol=1e-4, atol=1e-34)
    rtol, atol = (1e-4, 1e-5) if w.dtype == "fp32" else (2e-2, 1e-3)
    torch.testing.assert_close(out.float(), ref_out.float(), rtol=rtol, atol=atol)


def test_static_scratch_prefill_matches_oracle_and_regular_prefill_twice_in_a_row():
    from paper_2407_20485_b200 import binding as a2sf
    from paper_2407_20485_b200 import workloads as wl

    W = wl.WORKLOADS
    _case(a2sf, wl, W["llama2_7b"].scaled(H=4, n=700))                      # tensor-core passes
    _case(a2sf, wl, W["tiny_fp32"].scaled(n=100, budget=24, recent=8, alpha=0.9))   # CUDA-core passes
    # flags and score_window are honoured exactly as by a2sf_prefill
    _case(a2sf, wl, W["opt_6p7b"].scaled(B=1, H=2, n=300, alpha=0.9), score_window=64)
    _case(a2sf, wl, W["llama2_7b"].scaled(H=2, n=400, d=64), flags=a2sf.A2SF_FLAG_SKIP_ZERO_WEIGHT_ROWS)


def test_static_scratch_prefill_rejects_what_a2sf_prefill_rejects_and_oversized_calls():
    import ctypes

    from paper_2407_20485_b200 import binding as a2sf

    limit = int(a2sf.lib.a2sf_prefill_static_scratch_max_rows())
    assert limit == 1 << 20
    n = 4096
    H = limit // n + 1                       # one head too many
    q = torch.empty((1, 1, 8, 64), dtype=torch.bfloat16, device="cuda")   # never dereferenced
    fake = torch.empty((1, H, n, 64), dtype=torch.bfloat16, device="meta")

    def call(p):
        return a2sf.lib.a2sf_prefill_static_scratch(ctypes.byref(p), n, q.data_ptr(), q.data_ptr(), q.data_ptr(),
                                                    fake.stride(0), fake.stride(1), fake.stride(2),
                                                    q.data_ptr(), q.data_ptr(), q.data_ptr(), None)

    rc = call(a2sf.make_params(1, H, 64, torch.bfloat16, 32, 16, 0.5))
    assert rc == a2sf.A2SF_ERR_WORKSPACE
    assert "workspace" in a2sf.status_string(rc)
    assert call(a2sf.make_params(1, 2, 64, torch.bfloat16, 49153, 0, 0.5)) == a2sf.A2SF_ERR_UNSUPPORTED   # budget
    assert call(a2sf.make_params(1, 2, 64, torch.bfloat16, 32, 16, 0.5, flags=2)) == a2sf.A2SF_ERR_INVALID_ARG
    assert call(a2sf.make_params(1, 2, 64, torch.bfloat16, 32, 16, 0.5, score_window=-1)) == a2sf.A2SF_ERR_INVALID_ARG
