"""TEST INFRASTRUCTURE ONLY: the definitions behind paper_2502_02534_b200/selection.py, written out exactly.

pass@k (the paper's Eq. 1) with exact rational arithmetic and, for tiny n, by enumerating every k-subset; the
stratification by sorting and cutting, with the re-binning by boundary values done literally.
"""
from fractions import Fraction
from itertools import combinations
from math import comb


def pass_at_k_exact(n, correct, k):
    return sum(Fraction(1) - Fraction(comb(n - c, k), comb(n, k)) for c in correct) / len(correct)


def pass_at_k_enumerated(n, correct, k):
    """Fraction of k-subsets of n samples (the first c_i of them correct) that hold a correct one, averaged over tasks."""
    total = Fraction(0)
    for c in correct:
        hits = sum(1 for sub in combinations(range(n), k) if min(sub) < c)
        total += Fraction(hits, comb(n, k))
    return total / len(correct)


def stratify_literal(rates, m):
    """Section "Stratification and selection", step by step: sort ascending by success rate; lay the sorted list out
    as m consecutive runs whose sizes differ by at most one, the larger runs first (the reading of "as evenly as
    possible": the paper does not say where the remainder goes); the success rate of the first element of every run
    but the first is a boundary value; an experience's level is the number of boundary values it reaches."""
    n = len(rates)
    ranked = sorted(rates)
    runs, pos = [], 0
    for k in range(m):
        size = n // m + (1 if k < n % m else 0)
        runs.append(ranked[pos:pos + size])
        pos += size
    boundaries = []
    for run in runs[1:]:
        # an empty run (more levels than experiences) starts where the list ends: its boundary is the largest rate
        boundaries.append(run[0] if run else ranked[-1])
    levels = []
    for r in rates:
        lv = 0
        for b in boundaries:
            if r >= b:
                lv += 1
        levels.append(lv)
    return levels
