"""pass@k (Eq. 1) and the stratification beta: the host utilities against exact / enumerated definitions."""
import random
from fractions import Fraction

import pytest

from oracle import selection as ref
from paper_2502_02534_b200.selection import demonstrations, pass_at_k, stratify


def test_oracle_forms_agree_and_match_hand_values():
    # n = 4, c = 1, k = 2: 1 - C(3,2)/C(4,2) = 1 - 3/6
    assert ref.pass_at_k_exact(4, [1], 2) == Fraction(1, 2) == ref.pass_at_k_enumerated(4, [1], 2)
    for n in range(1, 7):
        for k in range(1, n + 1):
            cs = list(range(n + 1))
            assert ref.pass_at_k_exact(n, cs, k) == ref.pass_at_k_enumerated(n, cs, k)


def test_pass_at_k_extremes_and_random_cases():
    # pass@1 is the mean success rate, pass@n the share of tasks with at least one correct sample
    assert pass_at_k(64, [0, 16, 64], 1) == pytest.approx((0 + 0.25 + 1) / 3, abs=1e-15)
    assert pass_at_k(64, [0, 1, 64, 0], 64) == pytest.approx(0.5, abs=1e-15)
    rng = random.Random(0)
    for _ in range(200):
        n = rng.randint(1, 80); k = rng.randint(1, n)
        cs = [rng.randint(0, n) for _ in range(rng.randint(1, 26))]
        assert pass_at_k(n, cs, k) == pytest.approx(float(ref.pass_at_k_exact(n, cs, k)), abs=1e-12)
    assert pass_at_k(100000, [3], 50000) == pytest.approx(1 - 0.5 ** 3, rel=1e-4)   # no overflow at large n
    with pytest.raises(ValueError):
        pass_at_k(4, [5], 1)


def test_stratification_levels():
    rates = [0.9, 0.1, 0.5, 0.5, 0.2, 1.0]
    assert stratify(rates, 3) == [2, 0, 1, 1, 0, 2] == ref.stratify_literal(rates, 3)
    assert stratify(rates, 1) == [0] * 6
    # equal success rates share a level even when the even cut would separate them
    assert len(set(stratify([0.5] * 7, 3))) == 1
    rng = random.Random(1)
    for _ in range(200):
        rates = [rng.choice([0.0, 0.1, 0.25, 0.5, 0.75, 1.0]) for _ in range(rng.randint(1, 26))]
        m = rng.randint(1, 5)
        lv = stratify(rates, m)
        assert lv == ref.stratify_literal(rates, m)
        assert all(0 <= x < m for x in lv)
        for a in range(len(rates)):             # monotone in the success rate
            for b in range(len(rates)):
                if rates[a] < rates[b]:
                    assert lv[a] <= lv[b]
    lv = stratify([0.9, 0.1, 0.5], 3)
    assert demonstrations(lv, 0) == [1] and demonstrations(lv, 1) == [1, 2] and demonstrations(lv, 2) == [0, 1, 2]


def test_stratification_cut_positions_when_n_is_not_a_multiple_of_m():
    """Which runs take the remainder ("as evenly as possible" leaves it open; the reading is: the first n mod m runs,
    numpy.array_split's convention).  Hand-written levels of the sorted experiences, then numpy's own split."""
    import numpy as np
    distinct = lambda n: [i / 100 for i in range(n)]             # already ascending, all different
    assert ref.stratify_literal(distinct(7), 3) == [0, 0, 0, 1, 1, 2, 2] == stratify(distinct(7), 3)
    assert ref.stratify_literal(distinct(5), 4) == [0, 0, 1, 2, 3] == stratify(distinct(5), 4)
    assert ref.stratify_literal(distinct(6), 4) == [0, 0, 1, 1, 2, 3] == stratify(distinct(6), 4)   # ceil(k n / m) cuts would give [0,0,1,2,2,3]
    assert ref.stratify_literal(distinct(2), 4) == [0, 3] == stratify(distinct(2), 4)   # more levels than experiences: empty runs start at the end
    rng = random.Random(7)
    for _ in range(300):
        n, m = rng.randint(1, 40), rng.randint(1, 7)
        rates = rng.sample(range(1000), n)                        # distinct, shuffled
        expect = [0] * n
        order = sorted(range(n), key=lambda i: rates[i])
        for level, part in enumerate(np.array_split(np.array(order), m)):
            for i in part:
                expect[int(i)] = level
        if n >= m:        # with distinct rates and no empty run, re-binning by value changes nothing
            assert ref.stratify_literal(rates, m) == expect == stratify(rates, m)
        else:
            assert ref.stratify_literal(rates, m) == stratify(rates, m)
