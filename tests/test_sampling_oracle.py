"""Pins of the token-sampling oracle (oracle/sampling.py): the published known answers of its random number generator,
special cases that reduce to argmax, invariances, and the distribution the method must produce."""
import math
import os

import numpy as np

from oracle import sampling

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answer_vectors():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        got = sampling.philox4x32_10([np.array([x], dtype=np.uint32) for x in w[0:4]], [np.uint32(w[4]), np.uint32(w[5])])
        assert [int(g[0]) for g in got] == w[6:10]


def test_uniforms_lie_strictly_inside_the_unit_interval_and_streams_differ():
    u = sampling.uniforms(seed=7, step=3, row=5, vocab=10001)
    assert u.shape == (10001,) and (u > 0).all() and (u < 1).all()
    assert abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    for other in (sampling.uniforms(8, 3, 5, 10001), sampling.uniforms(7, 4, 5, 10001), sampling.uniforms(7, 3, 6, 10001),
                  sampling.uniforms(7 + (1 << 32), 3, 5, 10001)):
        assert (other != u).mean() > 0.99
    # index i only depends on (seed, step, row, i): a longer vocabulary extends the same stream
    assert np.array_equal(sampling.uniforms(7, 3, 5, 10)[:7], sampling.uniforms(7, 3, 5, 7))


def test_temperature_zero_is_argmax_with_ties_to_the_lowest_index():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6, 50))
    x[2, 10] = x[2, 30] = 9.0
    tok = sampling.sample_tokens(x, np.zeros(6), np.arange(6, dtype=np.uint64), step=0)
    assert np.array_equal(tok, np.argmax(x, axis=1)) and tok[2] == 10


def test_dominant_logit_always_wins_and_shifts_change_nothing():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((8, 33))
    seeds = np.arange(8, dtype=np.uint64) + 100
    T = np.full(8, 0.7)
    base = sampling.sample_tokens(x, T, seeds, step=2)
    assert np.array_equal(sampling.sample_tokens(x + 123.0, T, seeds, step=2), base)          # softmax is shift-invariant
    assert np.array_equal(sampling.sample_tokens(2 * x, 2 * T, seeds, step=2), base)          # only logits / T matters
    y = x.copy(); y[:, 4] = 1e4
    assert (sampling.sample_tokens(y, T, seeds, step=2) == 4).all()


def test_sampled_frequencies_follow_softmax_of_logits_over_temperature():
    """20000 independent draws (one seed each) over 6 tokens: the frequencies must match softmax(x / T) within 4.5 sigma;
    a missing logarithm, a wrong sign of the perturbation or temperature applied the wrong way round fails this."""
    x = np.array([1.0, 0.2, -0.5, 2.0, 0.0, -3.0])
    for T in (0.4, 1.0):
        p = np.exp(x / T - np.max(x / T)); p /= p.sum()
        n = 20000
        logits = np.broadcast_to(x, (n, 6))
        tok = sampling.sample_tokens(logits, np.full(n, T), np.arange(n, dtype=np.uint64) * 7919 + 11, step=0)
        freq = np.bincount(tok, minlength=6) / n
        sigma = np.sqrt(p * (1 - p) / n)
        assert (np.abs(freq - p) <= 4.5 * sigma + 1e-12).all(), (T, freq, p)
    # the rows of one call differ although the seeds are equal: the row index is part of the counter
    tok = sampling.sample_tokens(np.broadcast_to(x, (2000, 6)), np.full(2000, 1.0), np.full(2000, 5, dtype=np.uint64), step=0)
    assert len(set(tok.tolist())) >= 4
