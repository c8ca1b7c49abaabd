"""The seeded input generator: coordinate-addressed, reproducible, well distributed."""
import math

import numpy as np
import torch

from paper_2407_20485_b200 import workloads as wl


def _mix64_np(x):
    x = (x + np.uint64(0x9E3779B97F4A7C15))
    x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return x ^ (x >> np.uint64(31))


def test_mixer_matches_unsigned_reference():
    ctr = torch.arange(-5, 4000, dtype=torch.int64) * 7919
    got = wl._mix64(ctr).numpy().view(np.uint64)
    with np.errstate(over="ignore"):
        want = _mix64_np(ctr.numpy().view(np.uint64))
    np.testing.assert_array_equal(got, want)
    assert wl._mix64_int(12345) == int(_mix64_np(np.array([12345], dtype=np.uint64))[0])


def test_configs_match_the_stated_shapes():
    w = wl.WORKLOADS
    assert [x.index for x in w.values()] == [1, 2, 3, 4, 5]
    assert (w["llama2_7b"].budget, w["llama2_7b"].recent) == (205, 102)
    assert (w["opt_6p7b"].budget, w["opt_6p7b"].recent) == (205, 102)
    assert (w["llama2_13b"].B, w["llama2_13b"].H, w["llama2_13b"].n) == (32, 40, 4096)
    assert w["long_context"].alphas == (0.0, 0.5, 0.9, 1.0)
    # 2*512*128*2 + 12*512 + 6*128*2 + 16 bytes per head and step
    assert w["llama2_13b"].decode_bytes_per_unit_step() == 269_840
    assert w["tiny_fp32"].seed == 204851


def test_sub_blocks_equal_the_full_tensor():
    w = wl.WORKLOADS["tiny_fp32"]
    q, k, v = wl.make_prompt(w)
    assert q.shape == (1, 4, 128, 64) and q.dtype == torch.float32
    q2, k2, v2 = wl.make_prompt(w, h_range=(2, 3))
    assert torch.equal(q[:, 2:3], q2) and torch.equal(k[:, 2:3], k2) and torch.equal(v[:, 2:3], v2)
    qc, kc, vc = wl.make_prompt_chunked(w, "cpu", max_units_per_chunk=3)
    assert torch.equal(q, qc) and torch.equal(k, kc) and torch.equal(v, vc)
    dq, dk, dv = wl.make_decode(w)
    assert dq.shape == (16, 1, 4, 64)
    dq2, dk2, _ = wl.make_decode(w, t_range=(5, 9), h_range=(1, 4))
    assert torch.equal(dq[5:9, :, 1:4], dq2) and torch.equal(dk[5:9, :, 1:4], dk2)
    # reproducible
    q3, _, _ = wl.make_prompt(w)
    assert torch.equal(q, q3)


def test_heavy_hitters_and_distribution():
    w = wl.WORKLOADS["llama2_7b"].scaled(H=4)
    mask = wl.prompt_heavy_mask(w)
    assert mask[..., 0].all()
    assert (mask.sum(-1) == 1 + w.n_heavy).all()
    assert not torch.equal(mask[0, 0], mask[0, 1])             # per-head choice
    q, k, v = wl.make_prompt(w)
    qf = q.double()
    assert abs(qf.mean().item()) < 0.01 and abs(qf.std().item() - 1.0) < 0.01
    assert abs(v.double().std().item() - 1.0) < 0.01
    kstd_heavy = k.double()[mask].std().item()
    kstd_plain = k.double()[~mask].std().item()
    assert abs(kstd_heavy - 4.0) < 0.15 and abs(kstd_plain - 1.0) < 0.01
    # tensors are mutually independent draws
    assert abs((qf * v.double()).mean().item()) < 0.01
    t = wl.WORKLOADS["tiny_fp32"]
    assert (wl.prompt_heavy_mask(t).sum(-1) == 3).all()


def test_rounding_to_storage_dtype_is_exact_for_the_oracle():
    w = wl.WORKLOADS["llama2_7b"].scaled(H=1, n=64)
    q, _, _ = wl.make_prompt(w)
    assert q.dtype == torch.bfloat16
    # bf16 -> fp64 is exact, so both sides see the same numbers
    assert torch.equal(q.double().to(torch.bfloat16), q)


def test_shard_units_partitions_without_overlap():
    for total, ws in [(1280, 8), (32, 3), (4, 8), (7, 2)]:
        spans = [wl.shard_units(total, ws, r) for r in range(ws)]
        assert spans[0][0] == 0 and spans[-1][1] == total
        for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
            assert a1 == b0 and a0 <= a1
        sizes = [b - a for a, b in spans]
        assert max(sizes) - min(sizes) <= 1
