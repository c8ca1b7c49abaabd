"""Named cache policies as (alpha, budget, recent) triples.

The kernels take the three numbers directly; these helpers only fix the combinations the
paper discusses (Sec. 2.2, Sec. 4.1, Sec. 4.3):

* ``a2sf``  -- the paper's own setting: forgetting factor alpha in [0, 1), the whole budget is
  selective (no protected recent window);
* ``h2o``   -- plain accumulative score (alpha = 1), half of the budget reserved for the most
  recent tokens, half selected by score;
* ``local`` -- sliding window: the whole budget is the recent window, scores never decide.

``budget_for_ratio`` turns a cache ratio into a slot count the way the workloads do.
"""
from __future__ import annotations

import math
from dataclasses import dataclass


@dataclass(frozen=True)
class Policy:
    name: str
    alpha: float
    budget: int
    recent: int


def budget_for_ratio(ratio: float, n: int) -> int:
    """Slots for a cache ratio: ceil(ratio * n), at least 1."""
    if not (0.0 < ratio <= 1.0):
        raise ValueError("cache ratio must be in (0, 1]")
    return max(1, math.ceil(ratio * n - 1e-9))


def a2sf(budget: int, alpha: float = 0.3) -> Policy:
    if not (0.0 <= alpha <= 1.0):
        raise ValueError("alpha must be in [0, 1]")
    return Policy("a2sf", float(alpha), int(budget), 0)


def h2o(budget: int) -> Policy:
    return Policy("h2o", 1.0, int(budget), int(budget) // 2)


def local(budget: int) -> Policy:
    return Policy("local", 1.0, int(budget), int(budget))


def by_name(name: str, budget: int, alpha: float = 0.3) -> Policy:
    if name == "a2sf":
        return a2sf(budget, alpha)
    if name == "h2o":
        return h2o(budget)
    if name == "local":
        return local(budget)
    raise ValueError(f"unknown policy {name!r}")
