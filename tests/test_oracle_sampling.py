"""Pins of the oracle's counter-based generator and of its temperature sampler."""
import os

import numpy as np
import pytest

from oracle.accept import sample_token
from oracle.rng import philox4x32_10, step_uniform

KAT = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answer_vectors():
    rows = [l.split() for l in open(KAT) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        assert philox4x32_10(w[0:4], w[4:6]) == w[6:10]


def test_step_uniform_is_top_24_bits_and_depends_on_every_input():
    # counter (0, 0, 0, 0), key 0 -> first output word 0x6627e8d5 (first known-answer vector)
    assert step_uniform(0, 0, 0) == (0x6627E8D5 >> 8) / 2 ** 24
    base = step_uniform(5, 1, 7)
    assert 0.0 <= base < 1.0 and float(np.float32(base)) == base
    assert len({base, step_uniform(6, 1, 7), step_uniform(5, 2, 7), step_uniform(5, 1, 8),
                step_uniform(5 + (1 << 32), 1, 7)}) == 5


def test_sample_token_inverts_the_cdf_by_hand():
    # weights exp(z) = (1, 2, 1) at temperature 1: cumulative (1/4, 3/4, 1)
    z = np.log(np.array([1.0, 2.0, 1.0]))
    assert [sample_token(z, 1.0, u) for u in (0.0, 0.2499, 0.25, 0.5, 0.7499, 0.75, 0.9999)] == [0, 0, 1, 1, 1, 2, 2]
    # temperature 0.5 squares the weights: (1, 4, 1) / 6 -> boundaries 1/6 and 5/6
    assert [sample_token(z, 0.5, u) for u in (0.16, 0.17, 0.83, 0.84)] == [0, 1, 1, 2]
    # temperature 2 takes square roots: (1, 1.41421, 1) / 3.41421 -> boundaries 0.29289 and 0.70711
    assert [sample_token(z, 2.0, u) for u in (0.292, 0.294, 0.706, 0.708)] == [0, 1, 1, 2]
    # a token of zero weight is never drawn
    z2 = np.array([0.0, -np.inf, 0.0])
    assert {sample_token(z2, 1.0, u) for u in np.linspace(0, 0.999, 50)} == {0, 2}


def test_sampled_frequencies_on_a_four_token_vocabulary():
    """20000 draws through the generator follow softmax(z / T) within four binomial standard errors."""
    z, T, n = np.array([1.0, 0.0, -1.0, 2.0]), 0.8, 20000
    p = np.exp(z / T) / np.exp(z / T).sum()
    draws = np.array([sample_token(z, T, step_uniform(1234, 3, s)) for s in range(n)])
    freq = np.bincount(draws, minlength=4) / n
    assert np.all(np.abs(freq - p) < 4 * np.sqrt(p * (1 - p) / n))
    u = np.array([step_uniform(1234, 3, s) for s in range(n)])
    assert abs(u.mean() - 0.5) < 4 / np.sqrt(12 * n) and abs(np.mean(u < 0.1) - 0.1) < 4 * np.sqrt(0.09 / n)
