"""Seeded synthetic request streams shaped like the five benchmark configurations.

These stand in for the ShareGPT-v3 / guidellm streams the paper measures on
(Section 6.1), which are not available offline: only lengths, arrival
processes and sampling parameters are modelled; token ids are uniform random.
No arithmetic of the serving method lives here.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .configs import CONFIGS

STREAM_SEED_BASE = 0xB11C0000
# offered-load levels used for the rate sweep (13 levels between 1 and 32 req/s)
RATE_LEVELS = (1, 2, 3, 4, 5, 6, 7, 8, 10, 12, 16, 24, 32)


@dataclass
class Request:
    ticket: int
    arrival_s: float
    prompt: np.ndarray            # int32 [P]
    max_new: int
    top_k: int = 0                # 0 = greedy
    temperature: float = 1.0
    seed: int = 0
    eos_id: int = -1
    user_tag: int = 0
    top_p: float = 0.0            # outside (0, 1) = no nucleus cut
    extra: dict = field(default_factory=dict)

    @property
    def n_prompt(self) -> int:
        return int(self.prompt.shape[0])


def _lognormal_int(rng, median, sigma, lo, hi, n):
    x = np.exp(rng.normal(np.log(median), sigma, size=n))
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def make_requests(config: int, n_requests: int | None = None, rate: float | None = None,
                  seed: int | None = None, vocab: int | None = None) -> list[Request]:
    """Request stream of BASELINE configuration `config` (1..5)."""
    rng = np.random.default_rng((STREAM_SEED_BASE + config) if seed is None else seed)
    V = vocab if vocab is not None else CONFIGS[config]["model"].vocab
    if config == 1:
        n = n_requests or 8
        P = rng.integers(16, 65, size=n)
        N = np.full(n, 32)
        arr = np.zeros(n)
        topk, temp = 0, 1.0
    elif config == 2:
        n = n_requests or 128
        r = rate or 8.0
        P = rng.integers(128, 1025, size=n)
        N = rng.integers(128, 513, size=n)
        arr = np.cumsum(rng.exponential(1.0 / r, size=n))
        topk, temp = 0, 1.0
    elif config in (3, 4):
        n = n_requests or 512
        r = rate or 16.0
        P = _lognormal_int(rng, 512, 1.0, 4, 4096, n)
        N = _lognormal_int(rng, 256, 1.0, 4, 1024, n)
        arr = np.cumsum(rng.exponential(1.0 / r, size=n))
        topk, temp = 50, 0.8
    elif config == 5:
        n = n_requests or 256
        r = rate or 8.0
        P = rng.integers(256, 2049, size=n)
        N = rng.integers(128, 513, size=n)
        arr = np.cumsum(rng.exponential(1.0 / r, size=n))
        topk, temp = 0, 1.0
    else:
        raise ValueError(config)
    stream_seed = (STREAM_SEED_BASE + config) if seed is None else seed
    out = []
    for t in range(n):
        prompt = rng.integers(0, V, size=int(P[t]), dtype=np.int64).astype(np.int32)
        out.append(Request(ticket=t, arrival_s=float(arr[t]), prompt=prompt, max_new=int(N[t]),
                           top_k=topk, temperature=temp, seed=(stream_seed ^ t) & 0xFFFFFFFFFFFFFFFF,
                           user_tag=t))
    return out


def closed_batch(n: int, in_len: int, out_len: int, vocab: int, seed: int = 1,
                 top_k: int = 0, temperature: float = 1.0) -> list[Request]:
    """N x I -> O closed batch (all arrive at t = 0), the shape of the paper's
    scheduler-placement experiment (Fig. 3); gives clean fixed-batch decode steps."""
    rng = np.random.default_rng(seed)
    return [Request(ticket=t, arrival_s=0.0,
                    prompt=rng.integers(0, vocab, size=in_len, dtype=np.int64).astype(np.int32),
                    max_new=out_len, top_k=top_k, temperature=temperature,
                    seed=(seed * 7919 + t) & 0xFFFFFFFFFFFFFFFF, user_tag=t) for t in range(n)]
