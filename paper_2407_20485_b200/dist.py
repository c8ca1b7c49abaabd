"""Multi-process plumbing for the benchmark: one process per GPU, no data-path
collective.  (batch, head) units are independent, so ranks only meet at a barrier
and to combine their timings."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def _reduce(x: float, op, device) -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float, device="cpu") -> float:
    return _reduce(x, dist.ReduceOp.MAX, device)


def sum_over_ranks(x: float, device="cpu") -> float:
    return _reduce(x, dist.ReduceOp.SUM, device)


def rank_batch_range(per_gpu_batch: int, rank: int) -> Tuple[int, int]:
    """Weak scaling: every rank owns ``per_gpu_batch`` consecutive batch rows of a
    global workload whose batch is ``world_size * per_gpu_batch``."""
    return rank * per_gpu_batch, (rank + 1) * per_gpu_batch


def job_throughput(units_this_rank: float, ms_this_rank: float, device="cpu") -> Tuple[float, float]:
    """(total units over all ranks, max elapsed ms over ranks)."""
    return sum_over_ranks(units_this_rank, device), max_over_ranks(ms_this_rank, device)


def finalize():
    if dist.is_initialized():
        dist.destroy_process_group()
