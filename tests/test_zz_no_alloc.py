"""The allocation-free prefill entry point against the regular one.

Collected last on purpose (file name), so a run that stops at the first failure has
already exercised everything else.  Callers such as an inference engine whose own
pool allocator owns the GPU cannot call cudaMalloc; for them the library keeps the
prefill's log-sum-exp scratch in a fixed array of its device image.  The test calls
the entry point twice in a row with different shapes -- the second call finds the
first call's leftovers in the shared array -- and demands the regular entry
point's results both times.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(a2sf, wl, w):
    q, k, v = (t.cuda() for t in wl.make_prompt(w))
    p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha)
    ref_out, ref_S, ref_kept, _ = a2sf.a2sf_prefill(p, q, k, v)
    # the caller owns every buffer: allocate them before the call under test
    out = torch.empty_like(q)
    S = torch.empty_like(ref_S)
    kept = torch.empty_like(ref_kept)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    rc = a2sf.a2sf_prefill_static_scratch(p, q, k, v, out, S, kept)
    torch.cuda.synchronize()
    assert rc == a2sf.A2SF_OK, a2sf.status_string(rc)
    assert torch.cuda.memory_allocated() == before
    # same kernels, same order of operations: identical, well inside the parity
    # tolerances (scores 1e-4 relative, 16-bit outputs 2e-2 relative + 1e-3)
    assert torch.equal(kept, ref_kept)
    torch.testing.assert_close(S, ref_S, rtol=1e-4, atol=1e-34)
    torch.testing.assert_close(out.float(), ref_out.float(), rtol=2e-2, atol=1e-3)


def test_static_scratch_prefill_matches_regular_prefill_twice_in_a_row():
    from paper_2407_20485_b200 import binding as a2sf
    from paper_2407_20485_b200 import workloads as wl

    W = wl.WORKLOADS
    _case(a2sf, wl, W["llama2_7b"].scaled(H=4, n=700))
    _case(a2sf, wl, W["tiny_fp32"].scaled(n=100, budget=24, recent=8, alpha=0.9))


def test_static_scratch_prefill_rejects_oversized_calls():
    from paper_2407_20485_b200 import binding as a2sf

    limit = int(a2sf.lib.a2sf_prefill_static_scratch_max_rows())
    assert limit == 1 << 20
    n = 4096
    H = limit // n + 1                       # one head too many
    p = a2sf.make_params(1, H, 64, torch.bfloat16, 32, 16, 0.5)
    q = torch.empty((1, 1, 8, 64), dtype=torch.bfloat16, device="cuda")   # never dereferenced
    fake = torch.empty((1, H, n, 64), dtype=torch.bfloat16, device="meta")
    import ctypes

    rc = a2sf.lib.a2sf_prefill_static_scratch(ctypes.byref(p), n, q.data_ptr(), q.data_ptr(), q.data_ptr(),
                                              fake.stride(0), fake.stride(1), fake.stride(2),
                                              q.data_ptr(), q.data_ptr(), q.data_ptr(), None)
    assert rc == a2sf.A2SF_ERR_WORKSPACE
    assert "workspace" in a2sf.status_string(rc)
