"""Seeded synthetic workloads for the A2SF hot path.

This module holds the five workload descriptions and the coordinate-hashed
input generator.  It contains none of the method's arithmetic (no softmax, no
scores, no selection): it only produces Q/K/V tensors, so that the CPU oracle
and the CUDA library can be fed bit-identical inputs.

Every element is an independent N(0,1) draw that depends only on
``(seed, tensor, batch, head, token, channel)`` -- never on draw order -- so any
sub-block (one head, a few tokens) can be generated alone, on any device, and
equals the same block of the full tensor.

Heavy hitters (attention-sink / heavy-hitter structure of real decoder layers,
paper Sec. 2.2): per (batch, head), token 0 and a seeded set of further prompt
tokens have their K row multiplied by 4 before rounding to the storage dtype;
every decode token is heavy with probability 1 %.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import torch

# tensor identifiers mixed into the hash key
_TID_Q, _TID_K, _TID_V, _TID_HEAVY = 1, 2, 3, 4
_TID_DQ, _TID_DK, _TID_DV, _TID_DHEAVY = 5, 6, 7, 8

_DTYPES = {"fp32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16}
DTYPE_CODE = {"fp32": 0, "bf16": 1, "fp16": 2}
ELEM_BYTES = {"fp32": 4, "bf16": 2, "fp16": 2}

HEAVY_GAIN = 4.0
DECODE_HEAVY_PROB = 0.01


@dataclass(frozen=True)
class Workload:
    """One synthetic attention-layer workload (shapes + pruning policy)."""

    name: str
    index: int            # 1-based index of the configuration
    dtype: str            # "fp32" | "bf16" | "fp16"
    B: int
    H: int
    d: int
    n: int                # prompt length
    alpha: float
    budget: int           # M: cache slots per head
    recent: int           # R: protected newest positions
    steps: int            # T: decode steps
    n_heavy: int          # extra heavy prompt tokens besides token 0
    alphas: Tuple[float, ...] = ()   # forgetting-factor sweep (long-context case)

    @property
    def seed(self) -> int:
        return 204850 + self.index

    @property
    def units(self) -> int:
        return self.B * self.H

    @property
    def torch_dtype(self) -> torch.dtype:
        return _DTYPES[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return ELEM_BYTES[self.dtype]

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    def scaled(self, **kw) -> "Workload":
        """A copy with some fields replaced (shrunken parity-test variants)."""
        return replace(self, **kw)

    def decode_bytes_per_unit_step(self) -> int:
        """Algorithmic bytes one decode step moves for one (batch, head):
        K and V slots read, scores read + written, positions read, the three
        new vectors read, the output and the new K/V row written, plus the
        new score / position / evicted-slot / counters words."""
        M, d, e = self.budget, self.d, self.elem_bytes
        return 2 * M * d * e + 12 * M + 6 * d * e + 16

    def prefill_flops_per_unit(self) -> Dict[str, int]:
        """Causal (lower-triangle only) contraction flops per (batch, head)."""
        n, d = self.n, self.d
        return {"pass1": 2 * n * (n + 1) * d, "pass2": n * (n + 1) * d}


def _ceil_ratio(ratio_num: int, ratio_den: int, n: int) -> int:
    return -(-ratio_num * n // ratio_den)


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in (
        Workload("tiny_fp32", 1, "fp32", 1, 4, 64, 128, 0.5, 32, 16, 16, n_heavy=2),
        Workload("llama2_7b", 2, "bf16", 1, 32, 128, 1024, 0.3,
                 _ceil_ratio(1, 5, 1024), _ceil_ratio(1, 5, 1024) // 2, 256,
                 n_heavy=math.ceil(0.01 * 1024)),
        Workload("opt_6p7b", 3, "fp16", 8, 32, 128, 2048, 0.1,
                 _ceil_ratio(1, 10, 2048), _ceil_ratio(1, 10, 2048) // 2, 512,
                 n_heavy=math.ceil(0.01 * 2048)),
        Workload("llama2_13b", 4, "bf16", 32, 40, 128, 4096, 0.5, 512, 256, 512,
                 n_heavy=math.ceil(0.01 * 4096)),
        Workload("long_context", 5, "bf16", 1, 32, 128, 32768, 0.5, 2048, 1024, 1024,
                 n_heavy=math.ceil(0.01 * 32768), alphas=(0.0, 0.5, 0.9, 1.0)),
    )
}


# --------------------------------------------------------------------------
# counter-based generator: splitmix64 finaliser on int64 tensors (wrapping)
# --------------------------------------------------------------------------

def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit constant as signed (torch has no uint64 math)."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function (Steele, Lea, Flood 2014) on int64 bit patterns."""
    z = x + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _mix64_int(x: int) -> int:
    """The same mixer on a Python integer (used for keys)."""
    m = (1 << 64) - 1
    z = (x + 0x9E3779B97F4A7C15) & m
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    return z ^ (z >> 31)


def _key(seed: int, tensor_id: int, draw: int) -> int:
    return _s64(_mix64_int(_mix64_int(seed) ^ (tensor_id * 0x100 + draw)))


def _hash(seed: int, tensor_id: int, draw: int, counter: torch.Tensor) -> torch.Tensor:
    return _mix64(counter ^ _key(seed, tensor_id, draw))


def _uniform53(h: torch.Tensor) -> torch.Tensor:
    """Top 53 bits -> double in [0, 1)."""
    return _lsr(h, 11).to(torch.float64) * (1.0 / 9007199254740992.0)


def _normal(seed: int, tensor_id: int, counter: torch.Tensor) -> torch.Tensor:
    """Box-Muller N(0,1) in float64 from two hashed uniforms per element."""
    u1 = _uniform53(_hash(seed, tensor_id, 0, counter)) + (1.0 / 9007199254740992.0)
    u2 = _uniform53(_hash(seed, tensor_id, 1, counter))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def _counters(B_idx: torch.Tensor, H: int, h_idx: torch.Tensor, ntok: int,
              t_idx: torch.Tensor, d: int, device) -> torch.Tensor:
    """Element counter ((b*H + h)*ntok + t)*d + c, shape [b, h, t, d]."""
    c = torch.arange(d, dtype=torch.int64, device=device)
    unit = B_idx[:, None] * H + h_idx[None, :]                        # [b, h]
    row = unit[:, :, None] * ntok + t_idx[None, None, :]              # [b, h, t]
    return row[..., None] * d + c


def prompt_heavy_mask(w: Workload, device="cpu",
                      b_range: Optional[Tuple[int, int]] = None,
                      h_range: Optional[Tuple[int, int]] = None) -> torch.Tensor:
    """bool [b, h, n]: True where the prompt token's K row is heavy.

    Token 0 is always heavy; ``n_heavy`` further distinct tokens per (b, h) are
    the ones with the smallest hash among tokens 1..n-1."""
    b0, b1 = b_range or (0, w.B)
    h0, h1 = h_range or (0, w.H)
    bi = torch.arange(b0, b1, dtype=torch.int64, device=device)
    hi = torch.arange(h0, h1, dtype=torch.int64, device=device)
    ti = torch.arange(w.n, dtype=torch.int64, device=device)
    unit = bi[:, None] * w.H + hi[None, :]
    ctr = unit[:, :, None] * w.n + ti[None, None, :]
    hsh = _lsr(_hash(w.seed, _TID_HEAVY, 0, ctr), 1)                   # non-negative
    hsh[..., 0] = torch.iinfo(torch.int64).max                         # token 0 handled apart
    mask = torch.zeros(hsh.shape, dtype=torch.bool, device=device)
    k = min(w.n_heavy, w.n - 1)
    if k > 0:
        idx = torch.topk(hsh, k, dim=-1, largest=False).indices
        mask.scatter_(-1, idx, True)
    mask[..., 0] = True
    return mask


def make_prompt(w: Workload, device="cpu",
                b_range: Optional[Tuple[int, int]] = None,
                h_range: Optional[Tuple[int, int]] = None):
    """Q, K, V of shape [b, h, n, d] in the workload's dtype for a block of
    batches / heads (default: all)."""
    b0, b1 = b_range or (0, w.B)
    h0, h1 = h_range or (0, w.H)
    bi = torch.arange(b0, b1, dtype=torch.int64, device=device)
    hi = torch.arange(h0, h1, dtype=torch.int64, device=device)
    ti = torch.arange(w.n, dtype=torch.int64, device=device)
    ctr = _counters(bi, w.H, hi, w.n, ti, w.d, device)
    heavy = prompt_heavy_mask(w, device, (b0, b1), (h0, h1))
    gain = torch.where(heavy, HEAVY_GAIN, 1.0).to(torch.float64)[..., None]
    q = _normal(w.seed, _TID_Q, ctr).to(w.torch_dtype)
    k = (_normal(w.seed, _TID_K, ctr) * gain).to(w.torch_dtype)
    v = _normal(w.seed, _TID_V, ctr).to(w.torch_dtype)
    return q, k, v


def make_prompt_chunked(w: Workload, device, max_units_per_chunk: int = 64,
                        b_range: Optional[Tuple[int, int]] = None):
    """Full-size prompt tensors generated head-block by head-block so that the
    float64 intermediates stay small next to the result.  ``b_range`` selects a
    slice of the batch (one rank's share of a larger job)."""
    b0, b1 = b_range or (0, w.B)
    q = torch.empty((b1 - b0, w.H, w.n, w.d), dtype=w.torch_dtype, device=device)
    k = torch.empty_like(q)
    v = torch.empty_like(q)
    hstep = max(1, min(w.H, max_units_per_chunk))
    for b in range(b0, b1):
        for h0 in range(0, w.H, hstep):
            h1 = min(w.H, h0 + hstep)
            qq, kk, vv = make_prompt(w, device, (b, b + 1), (h0, h1))
            q[b - b0, h0:h1], k[b - b0, h0:h1], v[b - b0, h0:h1] = qq[0], kk[0], vv[0]
    return q, k, v


def make_decode(w: Workload, device="cpu",
                t_range: Optional[Tuple[int, int]] = None,
                b_range: Optional[Tuple[int, int]] = None,
                h_range: Optional[Tuple[int, int]] = None):
    """Decode-step inputs q, k_new, v_new of shape [t, b, h, d]."""
    t0, t1 = t_range or (0, w.steps)
    b0, b1 = b_range or (0, w.B)
    h0, h1 = h_range or (0, w.H)
    bi = torch.arange(b0, b1, dtype=torch.int64, device=device)
    hi = torch.arange(h0, h1, dtype=torch.int64, device=device)
    ti = torch.arange(t0, t1, dtype=torch.int64, device=device)
    c = torch.arange(w.d, dtype=torch.int64, device=device)
    unit = bi[:, None] * w.H + hi[None, :]                             # [b, h]
    row = ti[:, None, None] * w.units + unit[None]                     # [t, b, h]
    ctr = row[..., None] * w.d + c
    heavy = _uniform53(_hash(w.seed, _TID_DHEAVY, 0, row)) < DECODE_HEAVY_PROB
    gain = torch.where(heavy, HEAVY_GAIN, 1.0).to(torch.float64)[..., None]
    q = _normal(w.seed, _TID_DQ, ctr).to(w.torch_dtype)
    k = (_normal(w.seed, _TID_DK, ctr) * gain).to(w.torch_dtype)
    v = _normal(w.seed, _TID_DV, ctr).to(w.torch_dtype)
    return q, k, v


def shard_units(total_units: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous [lo, hi) slice of the (batch, head) units owned by ``rank``.
    Units are independent, so sharding needs no exchange step."""
    base, rem = divmod(total_units, world_size)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
