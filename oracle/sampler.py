"""Oracle O3: in-step token sampling.  TEST INFRASTRUCTURE ONLY.

The paper samples inside the captured step so that no host round trip happens
between the forward pass and next-token selection (Section 4.2, "CUDA graph
cache").  The two samplers the benchmark configurations use are written out:

  greedy : lowest index among the maxima of the row.
  top-k  : z = logit / T in IEEE fp32; keep the k largest by (z desc, index asc);
           w_j = exp(z_j - z_0) in fp64; u = (x >> 8) * 2^-24 with x the first
           word of Philox4x32-10(counter = {ticket_lo, ticket_hi, gen_index, 0},
           key = {seed_lo, seed_hi}); pick the smallest j with
           sum_{i<=j} w_i > u * sum_i w_i (sums taken left to right in fp64).

  top-p  : the sampler the paper names (Section 4.2, "CUDA graph cache": Top-P with
           temperature inside the step).  z and the order (z desc, index asc) as above, over
           the k largest when top_k > 0, else over the whole row.  Weights are integers so
           that no result depends on the order of a floating-point sum:
             q_j = floor(exp(z_j - z_0) * 2^40)        (exp in fp64, z_0 the largest z)
           With Q = sum_j q_j and P24 = round(top_p * 2^24) clamped to [1, 2^24], the nucleus
           is the smallest prefix j* of the order with  cum_j* * 2^24 >= P24 * Q; the draw is
           renormalised to it: with M = cum_j* and x24 = x >> 8 (the same Philox word x as
           top-k), pick the smallest j with cum_j > (x24 * M) >> 24.

Philox4x32-10 follows the published algorithm (Salmon et al., "Parallel random
numbers: as easy as 1, 2, 3", SC'11): ten rounds of two 32x32->64 multiplies with
the round key bumped by the Weyl constants.
"""
from __future__ import annotations

import numpy as np

_M0, _M1 = 0xD2511F53, 0xCD9E8D57
_W0, _W1 = 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """counter: 4 uint32, key: 2 uint32 -> 4 uint32 (python ints)."""
    c0, c1, c2, c3 = (int(c) & _MASK for c in counter)
    k0, k1 = (int(k) & _MASK for k in key)
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK
        hi1, lo1 = p1 >> 32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK, lo1, (hi0 ^ c3 ^ k1) & _MASK, lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def uniform_for(ticket: int, gen_index: int, seed: int) -> float:
    x = philox4x32_10((ticket & _MASK, (ticket >> 32) & _MASK, gen_index & _MASK, 0),
                      (seed & _MASK, (seed >> 32) & _MASK))[0]
    return (x >> 8) * 2.0 ** -24


def greedy(logits) -> int:
    row = np.asarray(logits)
    return int(np.flatnonzero(row == row.max())[0])


def top_k_candidates(logits, k: int, temperature: float):
    """(indices, z) of the k largest z = logit / T by (z desc, index asc); z is fp32."""
    z = (np.asarray(logits, dtype=np.float32) / np.float32(temperature)).astype(np.float32)
    order = np.lexsort((np.arange(z.shape[0]), -z.astype(np.float64)))[:k]
    return order, z[order]


def sample_top_k(logits, k: int, temperature: float, u: float) -> int:
    idx, z = top_k_candidates(logits, k, temperature)
    w = np.exp(z.astype(np.float64) - np.float64(z[0]))
    total = 0.0
    for x in w:
        total += float(x)
    thr = u * total
    acc = 0.0
    for j, x in enumerate(w):
        acc += float(x)
        if acc > thr:
            return int(idx[j])
    return int(idx[-1])


NUCLEUS_WEIGHT_BITS = 40


def philox_word(ticket: int, gen_index: int, seed: int) -> int:
    return philox4x32_10((ticket & _MASK, (ticket >> 32) & _MASK, gen_index & _MASK, 0),
                         (seed & _MASK, (seed >> 32) & _MASK))[0]


def nucleus(logits, k: int, temperature: float, top_p: float):
    """(indices, integer weights q) of the nucleus, in the order (z desc, index asc).
    k <= 0: the whole row is the candidate set."""
    n = len(logits)
    idx, z = top_k_candidates(logits, n if k <= 0 else min(k, n), temperature)
    w = np.exp(z.astype(np.float64) - np.float64(z[0]))
    q = [int(np.floor(x * float(1 << NUCLEUS_WEIGHT_BITS))) for x in w]     # python ints: exact sums
    Q = sum(q)
    p24 = min(max(int(np.rint(np.float64(np.float32(top_p)) * (1 << 24))), 1), 1 << 24)
    cum = 0
    for j, x in enumerate(q):
        cum += x
        if cum * (1 << 24) >= p24 * Q:
            return idx[: j + 1], q[: j + 1]
    return idx, q


def sample_top_p(logits, k: int, temperature: float, top_p: float, x24: int) -> int:
    idx, q = nucleus(logits, k, temperature, top_p)
    target = (x24 * sum(q)) >> 24
    cum = 0
    for j, x in enumerate(q):
        cum += x
        if cum > target:
            return int(idx[j])
    return int(idx[-1])


def sample(logits, top_k: int, temperature: float, ticket: int, gen_index: int, seed: int,
           top_p: float = 0.0) -> int:
    """top_p outside (0, 1) switches the nucleus off; then top_k <= 0 means greedy."""
    if 0.0 < top_p < 1.0:
        return sample_top_p(logits, top_k, temperature, top_p, philox_word(ticket, gen_index, seed) >> 8)
    if top_k <= 0:
        return greedy(logits)
    return sample_top_k(logits, min(top_k, len(logits)), temperature,
                        uniform_for(ticket, gen_index, seed))
