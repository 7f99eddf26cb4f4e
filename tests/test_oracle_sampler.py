"""Pins for the sampling oracle (Philox4x32-10, greedy, top-k)."""
import os

import numpy as np

from oracle import sampler as S

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    n = 0
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert list(S.philox4x32_10(w[0:4], w[4:6])) == w[6:10]
        n += 1
    assert n == 2


def test_philox_is_a_bijection_on_small_counters_and_key_sensitive():
    outs = {S.philox4x32_10((i, 0, 0, 0), (7, 9)) for i in range(2000)}
    assert len(outs) == 2000
    assert S.philox4x32_10((1, 2, 3, 0), (5, 6)) != S.philox4x32_10((1, 2, 3, 0), (5, 7))
    assert S.philox4x32_10((1, 2, 3, 0), (5, 6)) != S.philox4x32_10((1, 2, 4, 0), (5, 6))


def test_uniform_range_and_moments():
    u = np.array([S.uniform_for(3, i, 12345) for i in range(20000)])
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * (1 / 12 / 20000) ** 0.5
    assert abs(u.var() - 1 / 12) < 0.004


def test_greedy_lowest_index_among_maxima():
    assert S.greedy([1.0, 5.0, 5.0, 2.0]) == 1
    assert S.greedy([-np.inf, -3.0]) == 1


def test_topk_k1_and_small_temperature_equal_greedy():
    rng = np.random.default_rng(0)
    for i in range(50):
        row = rng.normal(size=97).astype(np.float32)
        g = S.greedy(row)
        assert S.sample(row, 1, 0.8, i, 0, 42) == g
        assert S.sample(row, 10, 1e-4, i, i, 42) == g


def test_topk_selection_matches_full_sort_with_ties():
    rng = np.random.default_rng(1)
    for _ in range(30):
        row = rng.integers(-3, 4, size=40).astype(np.float32)   # many exact ties
        idx, z = S.top_k_candidates(row, 7, 0.5)
        full = sorted(range(40), key=lambda i: (-(np.float32(row[i]) / np.float32(0.5)), i))[:7]
        assert list(idx) == full


def test_topk_frequencies_match_softmax():
    row = np.array([2.0, 1.0, 0.5, 0.0, -0.5, -1.0, -3.0, 1.5], dtype=np.float32)
    T, k, n = 0.8, 5, 100000
    idx, z = S.top_k_candidates(row, k, T)
    p = np.exp(z.astype(np.float64) - z[0])
    p /= p.sum()
    counts = np.zeros(8)
    for i in range(n):
        counts[S.sample(row, k, T, 11, i, 777)] += 1
    assert counts[[i for i in range(8) if i not in idx]].sum() == 0
    for j, i in enumerate(idx):
        sd = (n * p[j] * (1 - p[j])) ** 0.5
        assert abs(counts[i] - n * p[j]) < 4 * sd


def test_inverse_cdf_boundaries():
    row = np.array([0.0, 0.0, 0.0, 0.0], dtype=np.float32)     # equal weights 1/4 each
    assert S.sample_top_k(row, 4, 1.0, 0.0) == 0
    assert S.sample_top_k(row, 4, 1.0, 0.2499) == 0
    assert S.sample_top_k(row, 4, 1.0, 0.25) == 1              # needs sum > u*total, strictly
    assert S.sample_top_k(row, 4, 1.0, 0.9999) == 3
