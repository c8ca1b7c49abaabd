"""Policy presets (paper Sec. 4.1: H2O = half recent + half selected; A2SF = all selective)."""
import numpy as np
import pytest

from paper_2407_20485_b200 import policies


def test_preset_values():
    assert policies.a2sf(205, 0.3) == policies.Policy("a2sf", 0.3, 205, 0)
    assert policies.h2o(205) == policies.Policy("h2o", 1.0, 205, 102)
    assert policies.local(64) == policies.Policy("local", 1.0, 64, 64)
    assert policies.by_name("h2o", 10).recent == 5
    assert policies.budget_for_ratio(0.2, 1024) == 205 and policies.budget_for_ratio(0.1, 2048) == 205
    assert policies.budget_for_ratio(1.0, 7) == 7 and policies.budget_for_ratio(0.001, 10) == 1
    with pytest.raises(ValueError):
        policies.a2sf(8, 1.5)
    with pytest.raises(ValueError):
        policies.by_name("lru", 8)
    with pytest.raises(ValueError):
        policies.budget_for_ratio(0.0, 8)


def test_presets_differ_as_the_paper_describes_on_the_oracle():
    """On a sequence whose early tokens were attended long ago, H2O (alpha = 1) keeps them for
    their accumulated history while A2SF (alpha < 1) keeps what was attended recently (Sec. 3.2)."""
    import oracle

    rng = np.random.default_rng(0)
    n, d, M = 96, 16, 12
    K = rng.standard_normal((n, d))
    Q = rng.standard_normal((n, d))
    V = rng.standard_normal((n, d))
    early, late = 3, 70
    Q[4:48] += 3.0 * K[early]            # the first half of the queries looks at token `early`
    Q[72:] += 3.0 * K[late]              # the last quarter looks at token `late`
    scale = 1 / np.sqrt(d)
    kept = {}
    for pol in (policies.h2o(M), policies.a2sf(M, 0.3), policies.local(M)):
        res = oracle.prefill(Q[None], K[None], V[None], scale, [pol.alpha], pol.budget, pol.recent)
        kept[pol.name] = set(res["kept"][0].tolist())
    assert early in kept["h2o"] and late in kept["a2sf"]
    assert early not in kept["a2sf"]                         # forgotten: not attended recently
    assert kept["local"] == set(range(n - M, n))             # pure sliding window


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["a2sf", "h2o", "local"])
def test_presets_parity_on_gpu(name):
    from parity_util import run_parity
    from paper_2407_20485_b200 import workloads as wl

    base = wl.WORKLOADS["llama2_7b"]
    pol = policies.by_name(name, policies.budget_for_ratio(0.2, 600), alpha=0.3)
    w = base.scaled(H=2, n=600, steps=40, alpha=pol.alpha, budget=pol.budget, recent=pol.recent)
    rep = run_parity(w)
    assert rep.decode_evictions == 2 * 40
