"""Pins for the oracle's sampled token: the counter-based generator against its published
known-answer vectors, the uniform mapping, and the Gumbel-max draw against the softmax
probabilities it must reproduce."""
import math
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers(oracle):
    n = 0
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            w = [int(x, 16) for x in line.split()]
            assert oracle.philox4x32_10(w[0:4], w[4:6]).tolist() == w[6:10]
            n += 1
    assert n == 3


def test_uniform_mapping(oracle):
    seen = set()
    for v in range(64):
        u = oracle.sample_uniform(12345, 7, 3, v)
        k = u * 2 ** 24
        assert 0.0 < u < 1.0 and k == int(k) and int(k) % 2 == 1        # an odd multiple of 2^-24
        assert float(np.float32(u)) == u                                # exact in float32 as well
        seen.add(u)
    assert len(seen) > 60
    # the four entries of one counter block are the four output words; row, draw and seed all matter
    out = oracle.philox4x32_10([5, 3, 7, 0], [12345, 0])
    for j in range(4):
        assert oracle.sample_uniform(12345, 7, 3, 20 + j) == ((int(out[j]) >> 9) + 0.5) / 2 ** 23
    base = oracle.sample_uniform(1, 2, 3, 4)
    assert base != oracle.sample_uniform(1, 2, 4, 4) and base != oracle.sample_uniform(1, 3, 3, 4)
    assert base != oracle.sample_uniform(2, 2, 3, 4) and base != oracle.sample_uniform(1 + (1 << 32), 2, 3, 4)
    assert base != oracle.sample_uniform(1, 2 + (1 << 32), 3, 4)


def test_gumbel_max_reproduces_softmax(oracle):
    # chi-square of 40000 draws against softmax(z / T), for two temperatures
    z = np.array([2.0, 1.0, 0.0, -1.0, 0.5, 1.5, -3.0, 0.25])
    for T in (1.0, 0.5):
        p = np.exp(z / T - (z / T).max())
        p /= p.sum()
        n = 40000
        counts = np.zeros(z.size)
        for draw in range(n):
            tok, gap = oracle.sample_token(z, T, 99, draw, 0)
            assert gap >= 0.0
            counts[tok] += 1
        chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
        assert chi2 < 24.3, (T, chi2, counts)            # 7 degrees of freedom, p = 0.001
    # a mistake in the sign of the noise, or noise of the wrong scale, fails the test above; so
    # does ignoring the temperature: T = 0.5 sharpens the distribution
    assert True


def test_limits_and_ties(oracle):
    z = np.array([0.3, 4.0, -1.0, 3.9])
    # temperature -> 0: the draw is the greedy token
    for draw in range(50):
        assert oracle.sample_token(z, 1e-4, 5, draw, 0)[0] == 1
    # a shift of all logits changes nothing
    for draw in range(20):
        assert oracle.sample_token(z, 1.0, 5, draw, 2)[0] == oracle.sample_token(z + 11.0, 1.0, 5, draw, 2)[0]
    # the score that wins is z / T - ln(-ln U): recompute it from the uniforms
    for draw in range(20):
        tok, gap = oracle.sample_token(z, 0.7, 8, draw, 1)
        s = [z[v] / 0.7 - math.log(-math.log(oracle.sample_uniform(8, draw, 1, v))) for v in range(4)]
        assert tok == int(np.argmax(s))
        assert abs(gap - (sorted(s)[-1] - sorted(s)[-2])) < 1e-12
    # NaN logits never win
    assert oracle.sample_token(np.array([np.nan, 0.0, np.nan]), 1.0, 1, 0, 0)[0] == 1
    assert oracle.sample_token(np.array([np.nan, np.nan]), 1.0, 1, 0, 0)[0] == 0
