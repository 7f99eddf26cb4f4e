"""Oracle: the whole serving loop (O1 scheduling + O2 forward + O3 sampling) on the CPU.
TEST INFRASTRUCTURE ONLY.

Follows the request life cycle of the paper's Fig. 2 (steps 6-10): admitted
prompts are prefetched into the batch, each iteration runs one forward step
over the composed batch, samples in-step and publishes the tokens.
"""
from __future__ import annotations

import numpy as np

from . import sampler as S
from . import scheduler as O1
from . import transformer as O2


def run(model_cfg, sched, weights: O2.Weights, requests, watermarks=None, act_round=None,
        keep_logits=True, max_iters=10_000_000, forced=None, policy="chunked"):
    """requests: objects with ticket, prompt, max_new, top_k, temperature, seed, eos_id (and top_p, optional).
    forced: optional {ticket: [tokens]}: teacher forcing, the given tokens are fed back instead of
    the sampled ones (the sampled ones are still what `sampled` reports).
    Returns dict(trace, tokens {ticket: [fed-back tokens]}, sampled {ticket: [sampled tokens]},
    logits [(iter, bslot, ticket, gen_index, row)])."""
    sim = [O1.SimRequest(r.ticket, len(r.prompt), r.max_new, r.eos_id, r.prompt) for r in requests]
    byt = {r.ticket: r for r in requests}
    model = O2.PagedModel(model_cfg, weights, sched.n_blocks, sched.block_size, act_round)
    logs = []
    it_no = [0]
    sampled = {r.ticket: [] for r in requests}

    def sample_fn(items):
        lg = model.step(items)
        toks, row = [], 0
        for it in items:
            if not it.sample:
                continue
            r = byt[it.ticket]
            l32 = np.asarray(lg[row], dtype=np.float32)
            tok = S.sample(l32, r.top_k, r.temperature, r.ticket, it.gen_index, r.seed, getattr(r, "top_p", 0.0))
            sampled[it.ticket].append(tok)
            toks.append(tok if forced is None else int(forced[it.ticket][it.gen_index]))
            if keep_logits:
                logs.append((it_no[0], it.bslot, it.ticket, it.gen_index, np.array(lg[row])))
            row += 1
        it_no[0] += 1
        return toks

    trace, tokens, sch = O1.simulate(sim, sched.max_batch, sched.prefill_chunk_tokens,
                                     sched.n_blocks, sched.block_size, watermarks, sample_fn,
                                     max_iters=max_iters, policy=policy)
    return dict(trace=trace, tokens=tokens, sampled=sampled, logits=logs, scheduler=sch)
