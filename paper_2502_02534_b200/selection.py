"""Host-side numerics of the learning loop around the sampling step: pass@k (the paper's Eq. 1) and the
stratification beta of earned experience into m difficulty levels (section "Stratification and selection").
Integer / float work on a handful of tasks: plain Python, no device code.
"""
from __future__ import annotations

from typing import Sequence


def pass_at_k(n: int, correct: Sequence[int], k: int) -> float:
    """Eq. 1: mean over tasks of 1 - C(n - c_i, k) / C(n, k), with n samples per task and c_i correct ones.

    The ratio of binomials is evaluated as a running product, prod_{j = n-c+1}^{n} (1 - k / j), which stays in
    [0, 1] for any n (the binomials themselves overflow doubles beyond n ~ 1000)."""
    if not 1 <= k <= n:
        raise ValueError("need 1 <= k <= n")
    total = 0.0
    for c in correct:
        if not 0 <= c <= n:
            raise ValueError("need 0 <= c_i <= n")
        if n - c < k:
            total += 1.0          # every k-subset contains a correct sample
            continue
        miss = 1.0
        for j in range(n - c + 1, n + 1):
            miss *= 1.0 - k / j
        total += 1.0 - miss
    return total / len(correct) if len(correct) else 0.0


def stratify(success_rates: Sequence[float], m: int) -> list[int]:
    """beta's binning: level of every experience, 0 = hardest (lowest success rate) ... m-1 = easiest.

    Experiences are sorted by ascending success rate and cut into m runs of as equal size as possible; the success
    rates at the cuts become boundary VALUES, and every experience is then re-binned by value, so that equal success
    rates always share a level (a level may end up empty).

    "As evenly as possible" is read as: run sizes differ by at most one and the n mod m larger runs come FIRST (the
    hardest levels), the convention of numpy.array_split; the paper does not say which runs take the remainder."""
    n = len(success_rates)
    if m < 1:
        raise ValueError("need m >= 1")
    if n == 0:
        return []
    order = sorted(success_rates)
    q, r = divmod(n, m)
    starts = [k * q + min(k, r) for k in range(1, m)]          # index of the first element of run k
    boundaries = [order[min(n - 1, st)] for st in starts]
    return [sum(1 for b in boundaries if x >= b) for x in success_rates]


def demonstrations(levels: Sequence[int], j: int) -> list[int]:
    """Indices of the experiences in d_j = levels 0..j (selected incrementally: hard, hard+medium, ...)."""
    return [i for i, lv in enumerate(levels) if lv <= j]
