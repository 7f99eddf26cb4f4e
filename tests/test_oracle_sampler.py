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
    assert n == 3


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


# ---- top-p (nucleus) sampling: Section 4.2 names "Top-P with temperature" as the in-step sampler ----
def _softmax64(z):
    e = np.exp(z.astype(np.float64) - z.astype(np.float64).max())
    return e / e.sum()


def test_top_p_nucleus_is_the_smallest_prefix_reaching_p_brute_force():
    """Independent restatement in floating point on tiny rows: sort by probability, cut at the first
    prefix whose mass reaches p.  Rows whose cut lies within 1e-9 of p are skipped (the integer
    weights of the oracle and a float sum may then disagree legitimately)."""
    rng = np.random.default_rng(5)
    checked = 0
    for trial in range(200):
        n = int(rng.integers(2, 12))
        row = rng.normal(size=n).astype(np.float32) * 2
        T = float(rng.choice([0.5, 0.8, 1.0, 1.7]))
        p = float(rng.uniform(0.05, 0.99))
        z = (row / np.float32(T)).astype(np.float32)
        prob = _softmax64(z)
        order = sorted(range(n), key=lambda i: (-float(z[i]), i))
        cum = np.cumsum(prob[order])
        p_used = round(float(np.float32(p)) * 2 ** 24) / 2 ** 24
        if np.min(np.abs(cum - p_used)) < 1e-9:
            continue
        cut = int(np.argmax(cum >= p_used)) + 1
        idx, q = S.nucleus(row, 0, T, p)
        assert list(idx) == order[:cut]
        # the integer weights are the softmax numerators to 2^-40
        assert np.allclose(np.array(q, dtype=np.float64) / 2 ** 40, np.exp(z[order[:cut]].astype(np.float64) - float(z[order[0]])),
                           atol=2.0 ** -40)
        checked += 1
    assert checked > 150


def test_top_p_draw_follows_the_renormalised_inverse_cdf():
    rng = np.random.default_rng(6)
    for trial in range(100):
        row = rng.normal(size=9).astype(np.float32)
        idx, q = S.nucleus(row, 0, 0.9, 0.7)
        pr = np.array(q, dtype=np.float64) / float(sum(q))
        cum = np.cumsum(pr)
        x24 = int(rng.integers(0, 1 << 24))
        u = x24 / 2 ** 24
        if np.min(np.abs(cum - u)) < 1e-7:
            continue
        want = int(idx[int(np.argmax(cum > u))])
        assert S.sample_top_p(row, 0, 0.9, 0.7, x24) == want
    # boundaries: u = 0 takes the most likely token, the largest u the last of the nucleus
    row = np.array([0.0, 0.0, 0.0, 0.0], dtype=np.float32)
    assert S.sample_top_p(row, 0, 1.0, 0.75, 0) == 0
    assert S.sample_top_p(row, 0, 1.0, 0.75, (1 << 24) - 1) == 2      # nucleus = first three of four equal tokens
    assert S.sample_top_p(row, 0, 1.0, 0.76, (1 << 24) - 1) == 3      # 0.76 needs the fourth


def test_top_p_limits_equal_greedy_and_full_softmax_sampling():
    rng = np.random.default_rng(7)
    for i in range(40):
        row = rng.normal(size=61).astype(np.float32)
        assert S.sample(row, 0, 0.8, i, 3, 99, top_p=1e-6) == S.greedy(row)      # p -> 0: only the top token
    # p just below 1 keeps (numerically) the whole row: frequencies follow the full softmax
    row = np.array([2.0, 1.0, 0.5, 0.0, -0.5, -1.0, -3.0, 1.5], dtype=np.float32)
    T, n = 0.8, 60000
    pr = _softmax64((row / np.float32(T)).astype(np.float32))
    counts = np.zeros(8)
    for i in range(n):
        counts[S.sample(row, 0, T, 5, i, 2024, top_p=0.9999999)] += 1
    for i in range(8):
        assert abs(counts[i] - n * pr[i]) < 4 * (n * pr[i] * (1 - pr[i])) ** 0.5 + 1
    # top_p outside (0, 1) is "off": greedy when top_k is 0, plain top-k otherwise
    assert S.sample(row, 0, T, 1, 1, 1, top_p=1.0) == S.greedy(row)
    assert S.sample(row, 4, T, 1, 1, 1, top_p=0.0) == S.sample(row, 4, T, 1, 1, 1)


def test_top_p_frequencies_match_the_renormalised_nucleus_and_compose_with_top_k():
    row = np.array([2.0, 1.0, 0.5, 0.0, -0.5, -1.0, -3.0, 1.5], dtype=np.float32)
    T, p, n = 0.8, 0.8, 60000
    idx, q = S.nucleus(row, 0, T, p)
    pr = np.array(q, dtype=np.float64) / float(sum(q))
    counts = np.zeros(8)
    for i in range(n):
        counts[S.sample(row, 0, T, 21, i, 4242, top_p=p)] += 1
    assert counts[[i for i in range(8) if i not in idx]].sum() == 0
    for j, i in enumerate(idx):
        assert abs(counts[i] - n * pr[j]) < 4 * (n * pr[j] * (1 - pr[j])) ** 0.5
    # with top_k the nucleus is cut from the k largest only: same as top-p on the row restricted to them
    k = 3
    kidx, _ = S.top_k_candidates(row, k, T)
    sub = row[np.sort(kidx)]
    back = np.sort(kidx)
    for i in range(200):
        a = S.sample(row, k, T, 8, i, 17, top_p=0.6)
        b = back[S.sample(sub, 0, T, 8, i, 17, top_p=0.6)]
        assert a == b
