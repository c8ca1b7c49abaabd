"""The device-side failure path, exercised in the one form that cannot hang anything.

Every wait inside the library's kernels is bounded; a wait that runs out poisons its CTA, the
kernel unwinds and raises a sticky status word.  `a2sf_selftest_bounded_wait` runs that chain on
purpose and harmlessly: one CTA waits, through the library's own bounded wait with a short limit,
on a barrier nobody arrives at.  Nothing traps; the context stays usable.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu

LIMIT = 1_000_000          # SM clocks: about half a millisecond


@pytest.mark.parametrize("which", [0, 1])
def test_a_wait_that_runs_out_raises_the_sticky_status_once(which):
    from paper_2407_20485_b200 import binding as a2sf

    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK
    report = a2sf.a2sf_selftest_bounded_wait(which, LIMIT)
    torch.cuda.synchronize()                                   # the kernel returned: no hang, no trap
    failed, cycles, cycles_again, failed_again = report.cpu().tolist()
    assert failed == 1 and failed_again == 1
    assert LIMIT <= cycles < 40 * LIMIT                        # gave up after the limit, far below a second
    assert cycles_again < LIMIT // 10                          # a poisoned CTA does not spin again
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_ERR_TIMEOUT
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK      # reported once, then cleared
    assert "timed out" in a2sf.status_string(a2sf.A2SF_ERR_TIMEOUT)


def test_the_tensor_core_prefill_drains_while_the_status_is_set_and_works_again_after_the_clear():
    from paper_2407_20485_b200 import binding as a2sf
    from paper_2407_20485_b200 import workloads as wl
    from parity_util import run_parity

    w = wl.WORKLOADS["llama2_7b"].scaled(H=2, n=300, steps=4)
    q, k, v = wl.make_prompt(w, device="cuda")
    p = a2sf.make_params(w.B, w.H, w.d, w.torch_dtype, w.budget, w.recent, w.alpha)
    a2sf.a2sf_selftest_bounded_wait(0, LIMIT)
    # latched: the attention and scoring kernels return at once, so `out` keeps its sentinel
    out = torch.full_like(q, 7.0)
    a2sf.a2sf_prefill(p, q, k, v, out=out)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_ERR_TIMEOUT
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK
    # cleared: the same call now computes, and prefill + generation steps match the oracle
    a2sf.a2sf_prefill(p, q, k, v, out=out)
    torch.cuda.synchronize()
    assert not bool((out == 7.0).all())
    rep = run_parity(w)
    assert rep.decode_evictions == w.units * w.steps
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK


def test_the_generation_step_works_after_its_status_word_was_raised_and_cleared():
    from paper_2407_20485_b200 import binding as a2sf
    from paper_2407_20485_b200 import workloads as wl
    from parity_util import run_parity

    a2sf.a2sf_selftest_bounded_wait(1, LIMIT)
    torch.cuda.synchronize()
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_ERR_TIMEOUT
    w = wl.WORKLOADS["llama2_7b"].scaled(H=3, n=260, steps=6)
    rep = run_parity(w)
    assert rep.decode_evictions == w.units * w.steps
    assert a2sf.a2sf_last_device_status() == a2sf.A2SF_OK
