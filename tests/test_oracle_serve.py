"""Pins for oracle/serve.py::run (the whole loop on the CPU: scheduler + paged forward + sampler).

`run` only wires the three oracles together: which row belongs to which request, which token
index it samples, which tokens are fed back.  Pinned here against the unpaged dense forward of
each request taken alone (a request's output cannot depend on what else is in the batch)."""
import numpy as np

from oracle import sampler as S
from oracle import scheduler as O1
from oracle import serve as OS
from oracle import transformer as O2
from synth import make_requests, make_weights, model_cfg, sched_cfg, weights_as_numpy


def _setup(n_requests, **req_kw):
    model = model_cfg(1, dtype="fp32", n_layers=1, d_model=64, n_q_heads=2, n_kv_heads=1, head_dim=32, d_ff=128, vocab=257)
    sched = sched_cfg(1, prefill_chunk_tokens=24, max_batch=3, n_blocks=64)
    reqs = make_requests(1, n_requests=n_requests, vocab=model.vocab)
    for r in reqs:
        r.max_new = 6
        for k, v in req_kw.items():
            setattr(r, k, v)
    W = O2.Weights(model, weights_as_numpy(model, make_weights(model, 3, "cpu", random_gains=True)))
    return model, sched, reqs, W


def test_greedy_tokens_are_the_argmax_of_the_dense_forward_on_prompt_plus_own_tokens():
    model, sched, reqs, W = _setup(5)
    res = OS.run(model, sched, W, reqs)
    assert sorted(res["tokens"]) == [r.ticket for r in reqs]
    seen = set()
    for r in reqs:
        toks = res["tokens"][r.ticket]
        assert len(toks) == r.max_new
        seq = list(r.prompt) + toks[:-1]
        lg = O2.forward_dense(model, W, seq)
        for i in range(r.max_new):
            row = lg[r.n_prompt - 1 + i]
            assert toks[i] == int(np.argmax(row))
            margin = np.sort(row)[-1] - np.sort(row)[-2]
            assert margin > 1e-9          # the check above is not decided by rounding
    # every logged row is the row of that (ticket, index), equal to the dense forward
    for (it, bslot, ticket, gi, row) in res["logits"]:
        r = reqs[ticket]
        seq = list(r.prompt) + res["tokens"][ticket][:-1]
        want = O2.forward_dense(model, W, seq)[r.n_prompt - 1 + gi]
        assert np.abs(row - want).max() < 1e-9
        assert (ticket, gi) not in seen
        seen.add((ticket, gi))
        rec = res["trace"][it]
        assert (bslot, ticket) in [(s[0], s[1]) for s in rec["scheduled"]]
    assert len(seen) == sum(r.max_new for r in reqs)
    # three batch slots for five requests, chunked prompts: requests really shared steps
    assert max(len(rec["scheduled"]) for rec in res["trace"]) == 3


def test_sampled_tokens_use_the_requests_own_ticket_index_seed_and_fp32_logits():
    for kw in (dict(top_k=7, temperature=0.8), dict(top_k=0, temperature=0.9, top_p=0.8)):
        model, sched, reqs, W = _setup(4, **kw)
        for r in reqs:
            r.seed = 1000 + 17 * r.ticket
        res = OS.run(model, sched, W, reqs)
        for r in reqs:
            toks = res["tokens"][r.ticket]
            lg = O2.forward_dense(model, W, list(r.prompt) + toks[:-1])
            for i in range(r.max_new):
                row32 = np.asarray(lg[r.n_prompt - 1 + i], dtype=np.float32)   # the sampler sees fp32 logits
                assert toks[i] == S.sample(row32, r.top_k, r.temperature, r.ticket, i, r.seed, getattr(r, "top_p", 0.0))
        # a different seed changes some draw (the seed really reaches the sampler)
        reqs2 = [type(r)(**{**r.__dict__, "seed": r.seed + 1}) for r in reqs]
        res2 = OS.run(model, sched, W, reqs2)
        assert res2["tokens"] != res["tokens"]


def test_watermarks_and_eos_reach_the_scheduler():
    model, sched, reqs, W = _setup(3)
    full = OS.run(model, sched, W, reqs)
    # request 1 becomes visible only from iteration 2 on
    res = OS.run(model, sched, W, reqs, watermarks=[0, 0] + [2] * 200)
    assert [t for t, _ in res["trace"][0]["admitted"]] == [0] and res["trace"][1]["admitted"] == []
    assert res["tokens"] == full["tokens"]                     # outputs do not depend on arrival order
    # an EOS id that request 0 emits as its third token ends it there
    eos = full["tokens"][0][2]
    if eos not in full["tokens"][0][:2]:
        reqs[0].eos_id = eos
        cut = OS.run(model, sched, W, reqs)
        assert cut["tokens"][0] == full["tokens"][0][:3]
        assert cut["tokens"][1] == full["tokens"][1]


def test_teacher_forcing_feeds_the_given_tokens_and_still_reports_its_own_samples():
    model, sched, reqs, W = _setup(3)
    free = OS.run(model, sched, W, reqs)
    forced = {r.ticket: [(t + 1) % model.vocab for t in free["tokens"][r.ticket]] for r in reqs}
    res = OS.run(model, sched, W, reqs, forced=forced)
    assert res["tokens"] == forced                       # what was fed back
    for r in reqs:
        lg = O2.forward_dense(model, W, list(r.prompt) + forced[r.ticket][:-1])
        assert res["sampled"][r.ticket] == [int(np.argmax(lg[r.n_prompt - 1 + i])) for i in range(r.max_new)]
    assert free["sampled"] == free["tokens"]             # without forcing both are the same
