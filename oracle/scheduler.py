"""Oracle O1: iteration-level scheduler and paged-KV block allocator (integers, exact).

TEST INFRASTRUCTURE ONLY (see the package docstring).

What the paper fixes: continuous batching with first-come-first-served order
(Section 4.2, "Continuous batching with inline prefill"); new requests join a
running batch within one step; per-request progress is tracked so prefill can be
split into chunks (Section 7, "Serving optimizations"); slots move through
EMPTY -> PREFILL_PENDING -> PREFILL_PROCESSING -> DECODE_PROCESSING ->
DECODE_COMPLETED -> EMPTY (Section 4.2, "Ring buffer").  What it leaves open
(block size, admission rule, allocator) is fixed by the readings listed in the
design notes; this file is those readings written out step by step.

One iteration, given the watermark W (highest ticket visible to it):
  1. admit   - strictly by ascending ticket while a batch slot is free and
               reserved + need <= n_blocks, need = ceil((P + N - 1) / block);
               the admitted request takes the lowest free batch slot.
  2. compose - every DECODE request feeds one token (its last sampled token, at
               position P + generated - 1); then PREFILL requests in ascending
               ticket order take min(P - prefilled, budget_left) tokens, the
               budget starting at prefill_chunk_tokens each iteration.
  3. allocate- in ascending batch slot, pop ceil(new_len / block) - have blocks
               from the free stack (first pops of a fresh stack return 0, 1, 2...).
  4. forward + sample the rows that end a request's known tokens (every DECODE
               request; a PREFILL request whose chunk reaches P).
  5. post    - in ascending batch slot: append the token; at generated == N (or
               token == eos_id >= 0) push the blocks back in logical order,
               release the reservation and the batch slot.  Freed resources are
               usable from the next iteration.
Iterations that schedule nothing are not counted.

Second policy, "pause_resume": the paper's own inline prefill (Section 4.2, "Continuous
batching with inline prefill").  A step is either a decode step (every DECODE request feeds one
token) or a prefill step: the scheduler pauses the in-flight decode requests after the current
step (their slots are DECODE_PAUSED meanwhile), runs the whole prompts of the newly admitted
requests, merges them into the decode batch and resumes.  The paper's three conditions for
pausing are (i) pending prefills, (ii) free batch-slot capacity, (iii) launch-window headroom
for the prefill graph plus the resumed decode.  Here (i) and (ii) are the admission rule above;
(iii) belongs to the device-side graph-launch window, which the fused loop does not have, and is
always true.  Readings where the paper is silent: admitted prompts are taken whole, in ticket
order, while their total stays within the step's token capacity (never smaller than the longest
prompt, so the first always fits; nobody overtakes); a prefill step is followed by a decode step
whenever a DECODE request exists, so generation is paused for one step at a time.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Optional, Sequence

PREFILL = 1
DECODE = 2

# slot life cycle (Section 4.2, "Ring buffer")
EMPTY, PREFILL_PENDING, PREFILL_PROCESSING, DECODE_PROCESSING, DECODE_COMPLETED, DECODE_PAUSED = range(6)
LEGAL_TRANSITIONS = {
    (EMPTY, PREFILL_PENDING),
    (PREFILL_PENDING, PREFILL_PROCESSING),
    (PREFILL_PROCESSING, DECODE_PROCESSING),
    (DECODE_PROCESSING, DECODE_COMPLETED),
    (DECODE_COMPLETED, EMPTY),
    # a request whose only new token is produced by its last prefill chunk
    (PREFILL_PROCESSING, DECODE_COMPLETED),
    # pause-and-resume prefill: decode requests wait while new prompts are prefetched
    (DECODE_PROCESSING, DECODE_PAUSED),
    (DECODE_PAUSED, DECODE_PROCESSING),
    # a cancelled request is retired from wherever it stands (PREFILL_PROCESSING -> DECODE_COMPLETED is above)
    (DECODE_PAUSED, DECODE_COMPLETED),
}


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def blocks_needed(P: int, N: int, block: int) -> int:
    """Worst-case blocks of a request: positions 0 .. P+N-2 ever hold KV (the
    last sampled token is never fed back)."""
    return ceil_div(P + N - 1, block)


@dataclass
class SimRequest:
    ticket: int
    P: int
    N: int
    eos_id: int = -1
    prompt: Optional[Sequence[int]] = None


@dataclass
class _Entry:
    ticket: int
    P: int
    N: int
    eos_id: int
    need: int
    prefilled: int = 0
    generated: int = 0
    phase: int = PREFILL
    blocks: list = field(default_factory=list)
    tokens: list = field(default_factory=list)   # sampled so far


@dataclass
class ScheduledItem:
    bslot: int
    ticket: int
    phase: int
    start_pos: int
    n_tokens: int
    block_table: list          # physical ids, logical order, after this step's allocation
    sample: bool               # this item's last row is sampled
    gen_index: int             # index of the token that row samples
    input_tokens: Optional[list] = None   # filled when prompts are known


def fake_token(ticket: int, gen_index: int, vocab: int) -> int:
    """Deterministic stand-in sampler for control-only runs (no model math)."""
    x = (ticket * 2654435761 + gen_index * 40503 + 12345) & 0xFFFFFFFF
    return x % vocab


class Scheduler:
    """Incremental simulator.  `step(W)` runs one iteration and returns
    (trace_record, items) or None when nothing could be scheduled."""

    def __init__(self, requests: Sequence[SimRequest], max_batch: int, chunk: int,
                 n_blocks: int, block: int = 16, policy: str = "chunked"):
        assert policy in ("chunked", "pause_resume")
        self.policy = policy
        self.last_was_prefill = False
        self.req = {r.ticket: r for r in requests}
        self.MB, self.chunk, self.n_blocks, self.block = max_batch, chunk, n_blocks, block
        self.batch: list[Optional[_Entry]] = [None] * max_batch
        self.stack = list(range(n_blocks - 1, -1, -1))   # pop() returns 0, 1, 2, ...
        self.reserved = 0
        self.next_admit = min(self.req) if self.req else 0
        self.iter = 0
        self.slot_state = {t: PREFILL_PROCESSING for t in self.req}  # after claim
        self.transitions: list = []
        self._pending: Optional[dict] = None

    # -- step 1
    def _admit(self, W: int):
        admitted = []
        while self.next_admit <= W and self.next_admit in self.req:
            r = self.req[self.next_admit]
            free = [i for i, e in enumerate(self.batch) if e is None]
            need = blocks_needed(r.P, r.N, self.block)
            if not free or self.reserved + need > self.n_blocks:
                break          # head-of-line blocks: nobody overtakes
            b = free[0]
            self.batch[b] = _Entry(r.ticket, r.P, r.N, r.eos_id, need)
            self.reserved += need
            admitted.append((r.ticket, b))
            self.next_admit += 1
        return admitted

    # -- steps 1-3; returns None if nothing is schedulable
    def begin(self, W: int):
        assert self._pending is None
        admitted = self._admit(W)
        take = {}
        decoding = [b for b, e in enumerate(self.batch) if e is not None and e.phase == DECODE]
        prefilling = sorted((b for b, e in enumerate(self.batch) if e is not None and e.phase == PREFILL),
                            key=lambda b: self.batch[b].ticket)
        if self.policy == "chunked":
            for b in decoding:
                take[b] = 1
            budget = self.chunk
            for b in prefilling:
                if budget == 0:
                    break
                e = self.batch[b]
                n = min(e.P - e.prefilled, budget)
                take[b] = n
                budget -= n
        else:
            prefill_turn = bool(prefilling) and (not self.last_was_prefill or not decoding)
            if prefill_turn:
                room = self.chunk             # token capacity of a prefill step
                for b in prefilling:
                    e = self.batch[b]
                    if e.P > room:
                        break                 # whole prompts only, nobody overtakes
                    take[b] = e.P
                    room -= e.P
                for b in decoding:
                    if self.slot_state[self.batch[b].ticket] == DECODE_PROCESSING:
                        self._move(self.batch[b].ticket, DECODE_PAUSED)
            else:
                for b in decoding:
                    take[b] = 1
                    if self.slot_state[self.batch[b].ticket] == DECODE_PAUSED:
                        self._move(self.batch[b].ticket, DECODE_PROCESSING)
            if take:
                self.last_was_prefill = prefill_turn
        if not take:
            assert not admitted
            return None
        scheduled, allocated, items = [], [], []
        for b in sorted(take):
            e = self.batch[b]
            if e.phase == DECODE:
                start = e.P + e.generated - 1
            else:
                start = e.prefilled
            n = take[b]
            new_len = start + n
            want = ceil_div(new_len, self.block)
            while len(e.blocks) < want:
                blk = self.stack.pop()
                allocated.append((b, len(e.blocks), blk))
                e.blocks.append(blk)
            sample = (e.phase == DECODE) or (new_len == e.P)
            scheduled.append((b, e.ticket, e.phase, start, n))
            r = self.req[e.ticket]
            toks = None
            if e.phase == DECODE:
                toks = [e.tokens[-1]]
            elif r.prompt is not None:
                toks = [int(x) for x in r.prompt[start:start + n]]
            items.append(ScheduledItem(b, e.ticket, e.phase, start, n, list(e.blocks), sample,
                                       e.generated, toks))
        self._pending = dict(iter=self.iter, W=W, admitted=admitted, scheduled=scheduled,
                             allocated=allocated)
        return items

    # -- step 5
    def finish(self, items, sampled_tokens: Sequence[int], cancelled: Sequence[int] = ()):
        """`cancelled`: tickets whose cancellation the loop saw at the end of this iteration (the paper lists
        early exits among what the serving path must handle, Section 1; no mechanism is given): after the
        iteration's own completions, every live request among them is retired in ascending batch slot, its
        blocks pushed back in logical order and its reservation released, exactly as at a normal end."""
        rec = self._pending
        self._pending = None
        sampled, finished, freed = [], [], []
        it = iter(sampled_tokens)
        for item in items:
            e = self.batch[item.bslot]
            if e.phase == PREFILL:
                e.prefilled += item.n_tokens
            if not item.sample:
                continue
            tok = int(next(it))
            e.tokens.append(tok)
            e.generated += 1
            sampled.append((item.bslot, tok))
            if e.phase == PREFILL:
                e.phase = DECODE
                self._move(e.ticket, DECODE_PROCESSING if e.generated < e.N else DECODE_COMPLETED)
            if e.generated == e.N or (e.eos_id >= 0 and tok == e.eos_id):
                if self.slot_state[e.ticket] != DECODE_COMPLETED:
                    self._move(e.ticket, DECODE_COMPLETED)
                finished.append(e.ticket)
                for blk in e.blocks:
                    self.stack.append(blk)
                    freed.append(blk)
                self.reserved -= e.need
                self.batch[item.bslot] = None
        for b, e in enumerate(self.batch):
            if e is not None and e.ticket in cancelled:
                self._move(e.ticket, DECODE_COMPLETED)
                finished.append(e.ticket)
                for blk in e.blocks:
                    self.stack.append(blk)
                    freed.append(blk)
                self.reserved -= e.need
                self.batch[b] = None
        rec.update(sampled=sampled, finished=finished, freed=freed,
                   free_count=len(self.stack), reserved=self.reserved)
        self.iter += 1
        return rec

    def _move(self, ticket, new):
        old = self.slot_state[ticket]
        self.transitions.append((ticket, old, new))
        self.slot_state[ticket] = new

    @property
    def idle(self) -> bool:
        return all(e is None for e in self.batch)


def simulate(requests: Sequence[SimRequest], max_batch: int, chunk: int, n_blocks: int,
             block: int = 16, watermarks: Optional[Sequence[int]] = None,
             sample_fn: Optional[Callable] = None, vocab: int = 1 << 30,
             max_iters: int = 10_000_000, check: Optional[Callable] = None, policy: str = "chunked",
             cancels: Optional[dict] = None):
    """Run to drain.  `watermarks[i]` is W of traced iteration i (default: all
    requests visible from the start).  `sample_fn(items) -> tokens for the sample
    rows in order` (default: the control-only fake sampler).
    Returns (trace, tokens_by_ticket)."""
    sch = Scheduler(requests, max_batch, chunk, n_blocks, block, policy)
    last = max((r.ticket for r in requests), default=-1)
    trace, out = [], {r.ticket: [] for r in requests}
    while len(trace) < max_iters:
        W = last if watermarks is None else (watermarks[len(trace)] if len(trace) < len(watermarks) else None)
        if W is None:
            break
        items = sch.begin(W)
        if items is None:
            break
        if sample_fn is None:
            toks = [fake_token(i.ticket, i.gen_index, vocab) for i in items if i.sample]
        else:
            toks = sample_fn(items)
        rec = sch.finish(items, toks, (cancels or {}).get(len(trace), ()))
        for (b, tok), item in zip(rec["sampled"], [i for i in items if i.sample]):
            out[item.ticket].append(tok)
        trace.append(rec)
        if check is not None:
            check(sch)
    return trace, out, sch


# --------------------------------------------------------------------------------------
# Brute-force re-simulation: no incremental state.  Every iteration recomputes each
# request's progress, the batch-slot occupancy, the reservation and the free stack
# from the full history of decisions, straight from the definitions above.
# --------------------------------------------------------------------------------------
def brute_force(requests: Sequence[SimRequest], max_batch: int, chunk: int, n_blocks: int,
                block: int, watermarks: Sequence[int], tokens_by_ticket: dict):
    """Return the trace implied by the definitions, given the sampled tokens of
    every request (so it needs no sampler).  O(iterations * history)."""
    req = {r.ticket: r for r in requests}
    order = sorted(req)
    hist_admit = []      # (iter, ticket, bslot)
    hist_sched = []      # (iter, bslot, ticket, phase, start, n)
    hist_alloc = []      # (iter, ticket, logical, phys)
    hist_fin = []        # (iter, ticket)
    trace = []

    def prefilled(t):
        return sum(h[5] for h in hist_sched if h[2] == t and h[3] == PREFILL)

    def generated(t):
        r = req[t]
        g = 0
        for h in hist_sched:
            if h[2] != t:
                continue
            if h[3] == DECODE or h[4] + h[5] == r.P:
                g += 1
        return g

    def finished(t):
        return any(h[1] == t for h in hist_fin)

    def blocks_of(t):
        return [h[3] for h in sorted((h for h in hist_alloc if h[1] == t), key=lambda h: h[2])]

    def free_stack():
        # replay every pop and push in history order
        st = list(range(n_blocks - 1, -1, -1))
        # pops of an iteration come before its pushes; keep history order inside each kind
        pops = {}
        for it_, t, lg, ph in hist_alloc:
            pops.setdefault(it_, []).append(ph)
        pushes = {}
        for it_, t in hist_fin:
            pushes.setdefault(it_, []).append(t)
        for it_ in range(len(trace)):
            for ph in pops.get(it_, []):
                got = st.pop()
                assert got == ph
            for t in pushes.get(it_, []):
                # blocks the request held when it finished
                st.extend(h[3] for h in sorted((h for h in hist_alloc if h[1] == t and h[0] <= it_),
                                               key=lambda h: h[2]))
        return st

    for i, W in enumerate(watermarks):
        admitted_t = {h[1]: h[2] for h in hist_admit}
        live = {t: b for t, b in admitted_t.items() if not finished(t)}
        occupied = set(live.values())
        reserved = sum(blocks_needed(req[t].P, req[t].N, block) for t in live)
        # 1. admit
        admitted = []
        for t in order:
            if t in admitted_t:
                continue
            if t > W:
                break
            free = [b for b in range(max_batch) if b not in occupied]
            need = blocks_needed(req[t].P, req[t].N, block)
            if not free or reserved + need > n_blocks:
                break
            occupied.add(free[0])
            reserved += need
            live[t] = free[0]
            admitted.append((t, free[0]))
            hist_admit.append((i, t, free[0]))
        # 2. compose
        take = {}
        budget = chunk
        for t in sorted(live):
            r = req[t]
            pf = prefilled(t)
            if pf == r.P:
                take[t] = (DECODE, r.P + generated(t) - 1, 1)
        for t in sorted(live):
            r = req[t]
            pf = prefilled(t)
            if pf < r.P and budget > 0:
                n = min(r.P - pf, budget)
                budget -= n
                take[t] = (PREFILL, pf, n)
        if not take:
            break
        st = free_stack()
        scheduled, allocated, sampled, fin, freed = [], [], [], [], []
        new_sched = []
        for t in sorted(take, key=lambda t: live[t]):
            ph, start, n = take[t]
            b = live[t]
            have = len(blocks_of(t))
            for lg in range(have, ceil_div(start + n, block)):
                blk = st.pop()
                allocated.append((b, lg, blk))
                hist_alloc.append((i, t, lg, blk))
            scheduled.append((b, t, ph, start, n))
            new_sched.append((i, b, t, ph, start, n))
        # 5. post
        for (b, t, ph, start, n) in scheduled:
            r = req[t]
            if ph == DECODE or start + n == r.P:
                g = generated(t)          # before this iteration's row is recorded
                tok = tokens_by_ticket[t][g]
                sampled.append((b, tok))
                if g + 1 == r.N or (r.eos_id >= 0 and tok == r.eos_id):
                    fin.append(t)
        hist_sched.extend(new_sched)
        for t in fin:
            blks = blocks_of(t)
            st.extend(blks)
            freed.extend(blks)
            hist_fin.append((i, t))
            reserved -= blocks_needed(req[t].P, req[t].N, block)
        trace.append(dict(iter=i, W=W, admitted=admitted, scheduled=scheduled, allocated=allocated,
                          sampled=sampled, finished=fin, freed=freed, free_count=len(st),
                          reserved=reserved))
    return trace


def check_invariants(sch: Scheduler):
    """Allocator invariants that must hold after every iteration."""
    held = [b for e in sch.batch if e is not None for b in e.blocks]
    allb = held + sch.stack
    assert len(allb) == sch.n_blocks, "free + held must equal the pool"
    assert len(set(allb)) == sch.n_blocks, "a block is in exactly one place"
    assert len(held) <= sch.reserved <= sch.n_blocks
    assert sch.reserved == sum(e.need for e in sch.batch if e is not None)
    for e in sch.batch:
        if e is not None:
            assert len(e.blocks) <= e.need
