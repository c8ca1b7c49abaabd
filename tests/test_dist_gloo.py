"""The multi-process path on CPU (gloo, world_size 2): ranks own disjoint batch
slices of one global workload, meet only at barriers, and combine timings as
max-over-ranks / units as a sum."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _checksum(t):
    """Order-independent exact checksum of a float32 tensor's bit patterns."""
    return int(t.contiguous().view(torch.int32).to(torch.int64).sum().item())


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2407_20485_b200 import dist as a2dist
    from paper_2407_20485_b200 import workloads as wl

    r, lr, ws = a2dist.init("gloo")
    assert (r, ws) == (rank, world)
    w = wl.WORKLOADS["tiny_fp32"]
    wg = w.scaled(B=w.B * world)
    b_range = a2dist.rank_batch_range(w.B, rank)
    qk = wl.make_prompt_chunked(wg, "cpu", b_range=b_range)
    dq = wl.make_decode(wg, "cpu", b_range=b_range)
    a2dist.barrier()
    total_units, max_ms = a2dist.job_throughput(w.units, 10.0 * (rank + 1))
    lo, hi = wl.shard_units(wg.units, world, rank)
    q.put((rank, b_range, _checksum(qk[0]), _checksum(dq[0]), total_units, max_ms, (lo, hi),
           a2dist.sum_over_ranks(rank + 1.0)))
    a2dist.barrier()
    a2dist.finalize()


def test_two_ranks_share_one_global_workload():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    from paper_2407_20485_b200 import workloads as wl

    w = wl.WORKLOADS["tiny_fp32"]
    wg = w.scaled(B=2)
    full_q = wl.make_prompt(wg)[0]
    full_dq = wl.make_decode(wg)[0]
    for rank, b_range, qsum, dqsum, total_units, max_ms, span, ranksum in res:
        assert b_range == (rank, rank + 1)
        # each rank generated exactly its slice of the global tensors
        assert qsum == _checksum(full_q[rank:rank + 1])
        assert dqsum == _checksum(full_dq[:, rank:rank + 1])
        assert total_units == 2 * w.units          # whole-job units: sum over ranks
        assert max_ms == 20.0                      # elapsed: max over ranks
        assert span == (rank * w.units, (rank + 1) * w.units)
        assert ranksum == 3.0
    assert res[0][2] != res[1][2]                  # the slices differ


def test_single_process_helpers_without_a_group():
    from paper_2407_20485_b200 import dist as a2dist

    assert a2dist.max_over_ranks(3.5) == 3.5 and a2dist.sum_over_ranks(2.0) == 2.0
    a2dist.barrier()
    assert a2dist.rank_batch_range(32, 3) == (96, 128)
