"""Pins for the scheduler / block-allocator oracle: invariants, closed forms,
brute-force re-simulation, legal slot transitions."""
import numpy as np
import pytest

from oracle import scheduler as O1
from synth import make_requests


def _sim_reqs(reqs):
    return [O1.SimRequest(r.ticket, r.n_prompt, r.max_new) for r in reqs]


def _random_reqs(rng, n, pmax=70, nmax=20):
    return [O1.SimRequest(t, int(rng.integers(1, pmax)), int(rng.integers(1, nmax))) for t in range(n)]


def test_single_request_closed_form():
    for P, N, chunk in [(1, 1, 64), (16, 1, 64), (17, 5, 8), (64, 32, 64), (65, 3, 16), (130, 7, 64)]:
        tr, toks, sch = O1.simulate([O1.SimRequest(0, P, N)], 4, chunk, 64, 16, vocab=100)
        n_prefill = O1.ceil_div(P, chunk)
        assert len(tr) == n_prefill + N - 1
        assert sum(len(r["allocated"]) for r in tr) == O1.ceil_div(P + N - 1, 16)
        assert len(toks[0]) == N
        # physical ids come off a fresh stack as 0, 1, 2, ...
        assert [a[2] for r in tr for a in r["allocated"]] == list(range(O1.ceil_div(P + N - 1, 16)))
        assert tr[-1]["free_count"] == 64 and tr[-1]["reserved"] == 0


def test_max_batch_one_is_serial_in_ticket_order():
    rng = np.random.default_rng(3)
    reqs = _random_reqs(rng, 9)
    tr, toks, _ = O1.simulate(reqs, 1, 32, 64, 16, vocab=50)
    order = [t for r in tr for t in r["finished"]]
    assert order == list(range(9))
    for r in tr:
        assert len({s[1] for s in r["scheduled"]}) == 1
    assert len(tr) == sum(O1.ceil_div(q.P, 32) + q.N - 1 for q in reqs)


def test_conservation_and_invariants_random():
    rng = np.random.default_rng(5)
    for trial in range(20):
        reqs = _random_reqs(rng, int(rng.integers(1, 30)))
        nb = int(rng.integers(8, 40))
        reqs = [r for r in reqs if O1.blocks_needed(r.P, r.N, 16) <= nb]
        for i, r in enumerate(reqs):
            r.ticket = i
        mb = int(rng.integers(1, 9))
        chunk = int(rng.integers(1, 80))
        tr, toks, sch = O1.simulate(reqs, mb, chunk, nb, 16, vocab=1000, check=O1.check_invariants)
        assert sum(s[4] for r in tr for s in r["scheduled"] if s[2] == O1.PREFILL) == sum(q.P for q in reqs)
        assert sum(len(r["sampled"]) for r in tr) == sum(q.N for q in reqs)
        assert sorted(sch.stack) == list(range(nb)) and sch.reserved == 0
        for r in tr:
            assert sum(s[4] for s in r["scheduled"] if s[2] == O1.PREFILL) <= chunk
            assert len(r["scheduled"]) <= mb
            # token order inside a step: ascending batch slot
            assert [s[0] for s in r["scheduled"]] == sorted(s[0] for s in r["scheduled"])
        for (t, a, b) in sch.transitions:
            assert (a, b) in O1.LEGAL_TRANSITIONS


def test_fcfs_admission_order_and_head_of_line_blocking():
    # pool fits the big head request only after the first ones drain; the small one behind must wait
    reqs = [O1.SimRequest(0, 40, 8), O1.SimRequest(1, 100, 20), O1.SimRequest(2, 5, 2)]
    nb = 8     # need: 3, 8, 1
    tr, toks, _ = O1.simulate(reqs, 4, 64, nb, 16, vocab=10)
    adm = [(r["iter"], t) for r in tr for (t, b) in r["admitted"]]
    assert [t for _, t in adm] == [0, 1, 2]
    it0, it1, it2 = (i for i, _ in adm)
    fin0 = next(r["iter"] for r in tr if 0 in r["finished"])
    assert it1 == fin0 + 1            # freed resources usable from the next iteration
    assert it2 >= it1                 # never overtakes the blocked head
    fin1 = next(r["iter"] for r in tr if 1 in r["finished"])
    assert it2 == fin1 + 1            # pool is fully reserved by request 1 until it ends


def test_watermark_gates_visibility():
    reqs = [O1.SimRequest(t, 10, 3) for t in range(4)]
    W = [0, 0, 1, 3, 3, 3, 3, 3, 3]
    tr, _, _ = O1.simulate(reqs, 8, 64, 64, 16, watermarks=W, vocab=10)
    adm = {t: r["iter"] for r in tr for (t, b) in r["admitted"]}
    assert adm == {0: 0, 1: 2, 2: 3, 3: 3}


def test_lowest_free_batch_slot_and_lifo_block_reuse():
    reqs = [O1.SimRequest(0, 16, 2), O1.SimRequest(1, 16, 6), O1.SimRequest(2, 20, 2)]
    W = [1, 1, 2, 2, 2, 2, 2]
    tr, _, _ = O1.simulate(reqs, 4, 64, 16, 16, watermarks=W, vocab=10)
    assert tr[0]["admitted"] == [(0, 0), (1, 1)]
    assert tr[0]["allocated"] == [(0, 0, 0), (1, 0, 1)]
    # iteration 1: both decode at position 16 -> second block each: ids 2, 3; request 0 ends, frees 0 then 2
    assert tr[1]["allocated"] == [(0, 1, 2), (1, 1, 3)]
    assert tr[1]["finished"] == [0] and tr[1]["freed"] == [0, 2]
    # iteration 2: ticket 2 takes batch slot 0 again, pops the most recently pushed blocks first
    assert tr[2]["admitted"] == [(2, 0)]
    assert tr[2]["allocated"] == [(0, 0, 2), (0, 1, 0)]


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_brute_force_resimulation_agrees(seed):
    rng = np.random.default_rng(100 + seed)
    reqs = _random_reqs(rng, 12, pmax=60, nmax=9)
    nb, mb, chunk = 14, 3, int(rng.integers(5, 40))
    reqs = [r for r in reqs if O1.blocks_needed(r.P, r.N, 16) <= nb]
    for i, r in enumerate(reqs):
        r.ticket = i
    # a bursty visibility schedule
    W = []
    w = 0
    for i in range(400):
        if rng.random() < 0.3:
            w = min(len(reqs) - 1, w + int(rng.integers(1, 4)))
        W.append(w)
    tr, toks, _ = O1.simulate(reqs, mb, chunk, nb, 16, watermarks=W, vocab=64)
    bf = O1.brute_force(reqs, mb, chunk, nb, 16, W[:len(tr)], toks)
    assert len(bf) == len(tr)
    for a, b in zip(tr, bf):
        assert a == b


def test_eos_ends_a_request_early():
    r = O1.SimRequest(0, 5, 10, eos_id=7)
    seq = iter([1, 2, 7, 3, 4])
    tr, toks, sch = O1.simulate([r], 2, 64, 8, 16, sample_fn=lambda items: [next(seq) for i in items if i.sample])
    assert toks[0] == [1, 2, 7]
    assert sch.reserved == 0 and len(sch.stack) == 8


def test_config1_stream_shape_and_trace():
    reqs = make_requests(1)
    assert len(reqs) == 8 and all(16 <= r.n_prompt <= 64 and r.max_new == 32 for r in reqs)
    tr, toks, sch = O1.simulate(_sim_reqs(reqs), 8, 64, 256, 16, vocab=4096, check=O1.check_invariants)
    assert all(len(v) == 32 for v in toks.values())
    assert tr[0]["W"] == 7 and len(tr[0]["admitted"]) == 8


def test_config3_stream_trace_runs_at_full_scale():
    reqs = make_requests(3, n_requests=64)
    sim = _sim_reqs(reqs)
    tr, toks, sch = O1.simulate(sim, 256, 512, 60000, 16, vocab=128256)
    assert sum(len(v) for v in toks.values()) == sum(r.max_new for r in reqs)
    assert sch.reserved == 0 and len(sch.stack) == 60000


# ---- second policy: whole-prompt prefill with pause-and-resume (Section 4.2, "Continuous batching with
# inline prefill") -------------------------------------------------------------------------------------
def _pr(reqs, MB, cap, n_blocks, W=None, **kw):
    return O1.simulate(reqs, MB, cap, n_blocks, 16, watermarks=W, vocab=4096, policy="pause_resume",
                       check=O1.check_invariants, **kw)


def test_pause_resume_single_request_closed_form():
    for P, N in ((1, 1), (17, 5), (64, 32), (300, 2)):
        tr, toks, sch = _pr([O1.SimRequest(0, P, N)], 4, 512, 64)
        assert len(tr) == 1 + (N - 1)                                   # one whole-prompt step, then N - 1 decode steps
        assert tr[0]["scheduled"] == [(0, 0, O1.PREFILL, 0, P)]
        assert all(r["scheduled"] == [(0, 0, O1.DECODE, P + i, 1)] for i, r in enumerate(tr[1:]))
        assert len(toks[0]) == N and sch.idle and sch.reserved == 0


def test_pause_resume_steps_never_mix_phases_and_alternate():
    rng = np.random.default_rng(4)
    reqs = [O1.SimRequest(t, int(rng.integers(5, 120)), int(rng.integers(2, 30))) for t in range(24)]
    # arrivals trickle in: request t becomes visible at iteration 2 t
    W = [min(23, i // 2) for i in range(4000)]
    tr, toks, sch = _pr(reqs, 6, 160, 200, W=W)
    assert sch.idle and all(len(toks[r.ticket]) == r.N for r in reqs)
    kinds = []
    for rec in tr:
        ph = {s[2] for s in rec["scheduled"]}
        assert len(ph) == 1                                             # a step is a prefill step or a decode step
        kinds.append(ph.pop())
        if kinds[-1] == O1.PREFILL:
            assert all(s[3] == 0 and s[4] == reqs[s[1]].P for s in rec["scheduled"])   # whole prompts
            assert sum(s[4] for s in rec["scheduled"]) <= 160                          # within the step's capacity
            tk = [s[1] for s in sorted(rec["scheduled"], key=lambda s: s[1])]
            assert tk == list(range(tk[0], tk[0] + len(tk)))                           # consecutive tickets: nobody overtakes
    assert sum(s[4] for rec in tr for s in rec["scheduled"] if s[2] == O1.PREFILL) == sum(r.P for r in reqs)
    # generation is paused for one step at a time: two prefill steps in a row only while nothing decodes
    live_decode = set()
    for i, rec in enumerate(tr):
        if i > 0 and kinds[i] == O1.PREFILL and kinds[i - 1] == O1.PREFILL:
            assert not live_decode
        for s in rec["scheduled"]:
            if s[2] == O1.PREFILL and reqs[s[1]].N > 1:
                live_decode.add(s[1])
        for t in rec["finished"]:
            live_decode.discard(t)
    assert O1.PREFILL in kinds and O1.DECODE in kinds


def test_pause_resume_matches_a_restatement_from_history():
    """Every step is recomputed from the trace so far alone (no incremental state): which requests are
    admitted, prefetched, decoding or finished, whether the step before was a prefill step, and hence
    what this step must schedule."""
    rng = np.random.default_rng(12)
    for seed in range(4):
        n = 14
        reqs = [O1.SimRequest(t, int(rng.integers(3, 90)), int(rng.integers(1, 12))) for t in range(n)]
        W = sorted(int(x) for x in rng.integers(0, n, size=3000))
        MB, cap, nb = 4, 128, 40
        tr, toks, _ = _pr(reqs, MB, cap, nb, W=W)
        need = lambda r: O1.blocks_needed(r.P, r.N, 16)
        for i, rec in enumerate(tr):
            hist = tr[:i]
            admitted = {t: b for h in hist for (t, b) in h["admitted"]}
            finished = {t for h in hist for t in h["finished"]}
            prefilled = {s[1] for h in hist for s in h["scheduled"] if s[2] == O1.PREFILL}
            ngen = {t: sum(1 for h in hist for s in h["scheduled"] if s[1] == t) for t in admitted}
            live = {t: b for t, b in admitted.items() if t not in finished}
            reserved = sum(need(reqs[t]) for t in live)
            occupied = set(live.values())
            # admission
            exp_adm, nxt = [], len(admitted)
            while nxt < n and nxt <= W[i]:
                free = [b for b in range(MB) if b not in occupied]
                if not free or reserved + need(reqs[nxt]) > nb:
                    break
                exp_adm.append((nxt, free[0])); occupied.add(free[0]); live[nxt] = free[0]; reserved += need(reqs[nxt]); nxt += 1
            assert rec["admitted"] == exp_adm
            decoding = [t for t in live if t in prefilled]
            waiting = sorted(t for t in live if t not in prefilled)
            last_prefill = bool(hist) and hist[-1]["scheduled"][0][2] == O1.PREFILL
            if waiting and (not last_prefill or not decoding):
                exp, room = [], cap
                for t in waiting:
                    if reqs[t].P > room:
                        break
                    exp.append((live[t], t, O1.PREFILL, 0, reqs[t].P)); room -= reqs[t].P
            else:
                exp = [(live[t], t, O1.DECODE, reqs[t].P + ngen[t] - 1, 1) for t in decoding]
            assert sorted(rec["scheduled"]) == sorted(exp), (seed, i)


def test_pause_resume_slot_states_follow_the_paper_state_machine():
    reqs = [O1.SimRequest(t, 20 + t, 6) for t in range(6)]
    W = [0, 0, 0, 1, 1, 2, 2, 3, 4, 5] + [5] * 200
    tr, toks, sch = _pr(reqs, 3, 64, 64, W=W)
    assert all((a, b) in O1.LEGAL_TRANSITIONS for (_, a, b) in sch.transitions)
    paused = [(t, a, b) for (t, a, b) in sch.transitions if b == O1.DECODE_PAUSED]
    resumed = [(t, a, b) for (t, a, b) in sch.transitions if a == O1.DECODE_PAUSED]
    assert paused and len(paused) == len(resumed)                       # every pause is followed by a resume
    assert all(b == O1.DECODE_PROCESSING for (_, _, b) in resumed)


# ---- cancellation (an early exit the host asks for) ----------------------------------------------------
def test_cancel_retires_a_request_and_returns_everything_it_held():
    # alone: cancelled at the end of iteration 3 -> four iterations, all blocks back, nothing reserved
    tr, toks, sch = O1.simulate([O1.SimRequest(0, 40, 100)], 2, 64, 32, 16, vocab=4096, cancels={3: [0]},
                                check=O1.check_invariants)
    assert len(tr) == 4 and tr[3]["finished"] == [0] and len(toks[0]) == 4
    assert tr[3]["freed"] == [0, 1, 2] and tr[3]["free_count"] == 32 and tr[3]["reserved"] == 0 and sch.idle
    assert all((a, b) in O1.LEGAL_TRANSITIONS for (_, a, b) in sch.transitions)
    # in a full batch: the freed batch slot and blocks let the waiting request in one iteration later
    reqs = [O1.SimRequest(0, 30, 50), O1.SimRequest(1, 30, 50), O1.SimRequest(2, 20, 5)]
    base, _, _ = O1.simulate(reqs, 2, 64, 64, 16, vocab=4096, check=O1.check_invariants)
    cut, toks, _ = O1.simulate(reqs, 2, 64, 64, 16, vocab=4096, cancels={5: [1]}, check=O1.check_invariants)
    first_in = lambda tr: next(i for i, r in enumerate(tr) if any(t == 2 for t, _ in r["admitted"]))
    assert first_in(cut) == 6 and first_in(base) > 40
    assert cut[5]["finished"] == [1] and len(toks[1]) == 6 and len(toks[0]) == 50 and len(toks[2]) == 5
    assert cut[-1]["free_count"] == 64 and cut[-1]["reserved"] == 0
    # a ticket that is not live at that iteration (finished already, or not admitted yet) changes nothing
    same, _, _ = O1.simulate(reqs, 2, 64, 64, 16, vocab=4096, cancels={5: [2], 200: [0]})
    assert same == base
    # a request in the middle of a chunked prompt (no token yet) goes from PREFILL_PROCESSING to DECODE_COMPLETED
    tr, toks, sch = O1.simulate([O1.SimRequest(0, 200, 9)], 2, 64, 32, 16, vocab=4096, cancels={1: [0]})
    assert len(tr) == 2 and toks[0] == [] and (0, O1.PREFILL_PROCESSING, O1.DECODE_COMPLETED) in sch.transitions
