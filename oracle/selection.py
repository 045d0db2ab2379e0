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
    n = len(rates)
    order = sorted(range(n), key=lambda i: rates[i])
    # as even as possible: the first (n % m) runs hold one more ... cut points of the ceil-based even split
    cuts = [-(-k * n // m) for k in range(1, m)]
    boundaries = [rates[order[min(c, n - 1)]] for c in cuts]
    levels = []
    for r in rates:
        lv = 0
        for b in boundaries:
            if r >= b:
                lv += 1
        levels.append(lv)
    return levels
