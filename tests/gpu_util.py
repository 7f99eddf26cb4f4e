"""Helpers shared by the GPU parity tests: run a request stream through libblink and
through the oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import scheduler as O1
from oracle import serve as OS
from oracle import transformer as O2
from paper_2604_07609_b200 import binding as B
from synth import make_weights, weights_as_numpy


def sim_requests(reqs):
    return [O1.SimRequest(r.ticket, r.n_prompt, r.max_new, r.eos_id, r.prompt) for r in reqs]


def run_control_only(model, sched, reqs, *, exec_mode=B.EXEC_PERSISTENT, iteration_budget=0, trace_words=1 << 22,
                     submit_all_first=True, step_iters=8):
    """Control-only run (no model math).  Returns (parsed trace, tokens by ticket, stats)."""
    stepped = exec_mode == B.EXEC_STEPPED
    eng = B.Blink(model, sched, control_only=True, start_paused=True, exec_mode=exec_mode,
                  iteration_budget=iteration_budget, trace_words=trace_words, stats_iters=1 << 16,
                  idle_exit_us=300_000)
    try:
        for r in reqs:
            eng.submit_request(r)
        eng.blink_start()
        total = sum(r.max_new for r in reqs)
        ev = eng.drain(total, timeout_s=120, step_iters=step_iters if stepped else 0)
        if stepped:
            eng.blink_step(1)
        eng.blink_stop(final=False)
        st = eng.blink_get_stats()
        trace = B.parse_trace(eng.blink_get_trace())
        return trace, B.tokens_by_ticket(ev), st, eng.blink_get_iter_stats()
    finally:
        assert eng.blink_destroy() == B.BLINK_OK


def oracle_control_trace(sched, reqs, trace_gpu, vocab):
    W = [r["W"] for r in trace_gpu]
    tr, toks, _ = O1.simulate(sim_requests(reqs), sched.max_batch, sched.prefill_chunk_tokens, sched.n_blocks,
                              sched.block_size, watermarks=W, vocab=vocab)
    return tr, toks


def assert_traces_equal(a, b):
    assert len(a) == len(b), f"trace lengths differ: {len(a)} vs {len(b)}"
    for i, (x, y) in enumerate(zip(a, b)):
        for k in ("iter", "W", "admitted", "scheduled", "allocated", "sampled", "finished", "freed",
                  "free_count", "reserved"):
            xv = [tuple(v) if isinstance(v, (list, tuple)) else v for v in x[k]] if isinstance(x[k], list) else x[k]
            yv = [tuple(v) if isinstance(v, (list, tuple)) else v for v in y[k]] if isinstance(y[k], list) else y[k]
            assert xv == yv, f"iteration {i}, field {k}: {xv} != {yv}"


def oracle_run(model, sched, reqs, weights_cpu, act_round, dtype=np.float64):
    W = O2.Weights(model, weights_as_numpy(model, weights_cpu), dtype=dtype)
    return OS.run(model, sched, W, reqs, act_round=act_round)


def gpu_run_forced(model, sched, reqs, weights_cpu, forced, *, exec_mode=B.EXEC_PERSISTENT, gemm_impl=B.GEMM_AUTO,
                   capture_rows=None, step_iters=4, iteration_budget=0, weights_layout=B.WEIGHTS_ROW_MAJOR):
    """Teacher-forced run: request t is fed forced[t] but reports its own samples.
    Returns (trace, sampled tokens by ticket, captured logits [rows, V] as numpy)."""
    dev = torch.device("cuda:0")
    wd = weights_cpu.to(dev)
    if weights_layout != B.WEIGHTS_ROW_MAJOR:
        B.blink_convert_weights(model, wd, B.WEIGHTS_ROW_MAJOR, weights_layout)
    kv = torch.zeros(sched.n_blocks * B.kv_bytes_per_block(model, sched.block_size), dtype=torch.uint8, device=dev)
    total = sum(r.max_new for r in reqs)
    cap = torch.zeros((capture_rows or total, model.vocab), dtype=torch.float32, device=dev)
    stepped = exec_mode == B.EXEC_STEPPED
    eng = B.Blink(model, sched, wd, kv, start_paused=True, exec_mode=exec_mode, gemm_impl=gemm_impl,
                  trace_words=1 << 22, stats_iters=1 << 14, logits_capture=cap, idle_exit_us=300_000,
                  iteration_budget=iteration_budget, weights_layout=weights_layout)
    try:
        for r in reqs:
            eng.submit_request(r, forced_tokens=None if forced is None else forced[r.ticket])
        eng.blink_start()
        ev = eng.drain(total, timeout_s=300, step_iters=step_iters if stepped else 0)
        if stepped:
            eng.blink_step(1)
        eng.blink_stop(final=False)
        trace = B.parse_trace(eng.blink_get_trace())
        st = eng.blink_get_stats()
        assert st.device_status == 0, f"device status {st.device_status}"
        torch.cuda.synchronize()
        return trace, B.tokens_by_ticket(ev), cap.cpu().numpy(), eng.blink_get_iter_stats()
    finally:
        assert eng.blink_destroy() == B.BLINK_OK


# ---- token rules near ties (a decision that rounding inside the tolerance may flip) -----------------
def acceptable_tokens(row, req, gen_index, tol):
    """Tokens a correct implementation may emit for oracle logits `row` when its own logits are
    within `tol` (max-abs) of them.  Greedy: every token within 2*tol of the maximum.  Top-k /
    top-p: the oracle's token, plus the neighbouring candidates when the draw lies within the
    distance by which a tol-perturbation can move an inverse-CDF boundary, plus the entries at a
    candidate-set boundary that is itself inside the margin.  Returns (set, in_margin)."""
    from oracle import sampler as S
    row = np.asarray(row, dtype=np.float32)
    top_p = getattr(req, "top_p", 0.0)
    nucleus_on = 0.0 < top_p < 1.0
    if req.top_k <= 0 and not nucleus_on:
        mx = float(row.max())
        ok = set(int(i) for i in np.flatnonzero(row >= mx - 2 * tol))
        return ok, len(ok) > 1
    want = S.sample(row, req.top_k, req.temperature, req.ticket, gen_index, req.seed, top_p)
    T = float(req.temperature)
    n = len(row)
    k = n if req.top_k <= 0 else min(req.top_k, n)
    idx, z = S.top_k_candidates(row, min(n, k + 1), T)
    ok, in_margin = {want}, False
    if k < n and float(z[k - 1]) - float(z[k]) < 2 * tol / T:       # the k-th and (k+1)-th candidates may swap
        in_margin = True
        ok.update(int(i) for i in idx[max(0, k - 2):k + 1])
    idx, z = idx[:k], z[:k].astype(np.float64)
    w = np.exp(z - z[0])
    if nucleus_on:
        nidx, _ = S.nucleus(row, req.top_k, T, top_p)
        m = len(nidx)
        cfrac = np.cumsum(w) / w.sum()
        d = 4 * tol / T + 1e-7
        if m < k and abs(cfrac[m - 1] - top_p) < d or (m >= 2 and abs(cfrac[m - 2] - top_p) < d):
            in_margin = True                                           # the nucleus may gain or lose its last token
            ok.update(int(i) for i in idx[:min(k, m + 1)])
            return ok, in_margin
        w, idx = w[:m], idx[:m]
    cfrac = np.cumsum(w) / w.sum()
    u = (S.philox_word(req.ticket, gen_index, req.seed) >> 8) / 2.0 ** 24
    j = int(np.flatnonzero(idx == want)[0])
    d = 4 * tol / T + 1e-7
    if j > 0 and u - cfrac[j - 1] < d:
        in_margin = True
        ok.add(int(idx[j - 1]))
    if j + 1 < len(idx) and cfrac[j] - u < d:
        in_margin = True
        ok.add(int(idx[j + 1]))
    return ok, in_margin


def assert_tokens_within_margin(ora, reqs, toks_gpu, tol):
    """Under teacher forcing the sampled token of every (ticket, index) must be the oracle's, except
    where the oracle's own decision margin is inside the tolerance; there it must be one of the
    in-margin candidates.  Returns the number of in-margin decisions."""
    by_ticket = {r.ticket: r for r in reqs}
    n_margin = 0
    for (_, _, ticket, gi, row) in ora["logits"]:
        ok, im = acceptable_tokens(row, by_ticket[ticket], gi, tol)
        n_margin += int(im)
        got = toks_gpu[ticket][gi]
        assert got in ok, f"ticket {ticket} index {gi}: token {got} not among the admissible {sorted(ok)[:8]}"
        if not im:
            assert got == ora["sampled"][ticket][gi]
    return n_margin


def compare_with_oracle(model, sched, reqs, weights_cpu, tol, *, oracle_dtype=np.float64, plain_too=True, **kw):
    """The whole check of one configuration: the oracle in the data path's rounding mode runs free
    (its own tokens fed back); the GPU is teacher-forced with those tokens; traces must be equal word
    for word (sampled tokens apart), logits within `tol`, tokens by the margin rule.  For the bf16 data
    path the plain high-precision oracle (no rounding hook) is run on the same forced tokens as well
    and the error against it reported."""
    matched_round = O2.round_bf16 if model.dtype == "bf16" else None
    W = O2.Weights(model, weights_as_numpy(model, weights_cpu), dtype=oracle_dtype)
    ora = OS.run(model, sched, W, reqs, act_round=matched_round)
    trace, toks, logits, its = gpu_run_forced(model, sched, reqs, weights_cpu, ora["tokens"], **kw)
    assert_traces_equal([{**r, "sampled": []} for r in trace], [{**r, "sampled": []} for r in ora["trace"]])
    lo = np.stack([row for (_, _, _, _, row) in ora["logits"]])
    assert logits.shape == lo.shape
    err = float(np.abs(logits.astype(np.float64) - lo).max())
    assert err <= tol, f"max-abs logit error {err:.3e} against the oracle exceeds {tol}"
    n_margin = assert_tokens_within_margin(ora, reqs, toks, tol)
    err_plain = err
    if plain_too and matched_round is not None:
        plain = OS.run(model, sched, W, reqs, act_round=None, forced=ora["tokens"])
        lp = np.stack([row for (_, _, _, _, row) in plain["logits"]])
        err_plain = float(np.abs(logits.astype(np.float64) - lp).max())
    return dict(err=err, err_plain=err_plain, n_margin=n_margin, trace=trace, toks=toks, ora=ora, its=its, logits=logits)
