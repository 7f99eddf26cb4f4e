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
                     submit_all_first=True, step_iters=8, policy=B.POLICY_CHUNKED, trickle=0):
    """Control-only run (no model math).  Returns (parsed trace, tokens by ticket, stats)."""
    stepped = exec_mode == B.EXEC_STEPPED
    eng = B.Blink(model, sched, control_only=True, start_paused=True, exec_mode=exec_mode,
                  iteration_budget=iteration_budget, trace_words=trace_words, stats_iters=1 << 16,
                  idle_exit_us=300_000, policy=policy)
    try:
        import time
        for r in reqs[:len(reqs) - trickle]:
            eng.submit_request(r)
        eng.blink_start()
        for r in reqs[len(reqs) - trickle:]:      # the rest arrive while the loop runs (watermarks are logged)
            time.sleep(0.0005)
            eng.submit_request(r)
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


def oracle_control_trace(sched, reqs, trace_gpu, vocab, policy="chunked"):
    W = [r["W"] for r in trace_gpu]
    tr, toks, _ = O1.simulate(sim_requests(reqs), sched.max_batch, sched.prefill_chunk_tokens, sched.n_blocks,
                              sched.block_size, watermarks=W, vocab=vocab, policy=policy)
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
                   capture_rows=None, step_iters=4, iteration_budget=0, weights_layout=B.WEIGHTS_ROW_MAJOR,
                   epilogue_fusion=B.FUSION_AUTO, policy=B.POLICY_CHUNKED):
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
                  iteration_budget=iteration_budget, weights_layout=weights_layout, epilogue_fusion=epilogue_fusion,
                  policy=policy)
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
    z_all = (row / np.float32(T)).astype(np.float32)
    idx, z = S.top_k_candidates(row, k, T)
    zs = z.astype(np.float64)
    tail_pool, p0, d_set = None, k, 0.0
    if k < n:
        # candidate set: a token whose z is within the margin of the k-th largest may be a member of the
        # other side's top k.  Then the positions from the first oracle member that may drop out (p0) to
        # the end may hold any of those members or of the outsiders that may come in, and the total mass
        # is uncertain by the mass of those positions.
        wide = np.flatnonzero(z_all >= z[k - 1] - 2 * tol / T)
        if len(wide) > k:
            p0 = int(np.argmax(zs < zs[k - 1] + 2 * tol / T))
            tail_pool = set(int(i) for i in wide if z_all[i] < zs[k - 1] + 2 * tol / T)
    w = np.exp(zs - zs[0])
    idx_all, zs_all = idx, zs
    d = float(np.expm1(2 * tol / T)) + 1e-7      # how far a tol-perturbation can move a normalised cumulative sum
    if tail_pool is not None:
        d += float(w[p0:].sum() / w.sum())
    cf = np.cumsum(w) / w.sum()
    prev = np.concatenate([[0.0], cf[:-1]])
    m_lo = m_hi = len(cf)
    if nucleus_on:   # the nucleus ends at the first prefix reaching top_p; the other side's may end a little earlier or later
        m_lo = min(len(cf), int(np.argmax(cf >= top_p - d)) + 1) if (cf >= top_p - d).any() else len(cf)
        m_hi = min(len(cf), int(np.argmax(cf >= top_p + d)) + 1) if (cf >= top_p + d).any() else len(cf)
    u = (S.philox_word(req.ticket, gen_index, req.seed) >> 8) / 2.0 ** 24
    # the draw lands at u * (mass of the nucleus); masses and boundaries each move by at most d
    t_lo, t_hi = u * (cf[m_lo - 1] - d), u * (cf[m_hi - 1] + d)
    pos = np.arange(len(cf))
    hit = np.flatnonzero((pos < m_hi) & (prev - d <= t_hi) & (cf + d >= t_lo))
    ok = {want}
    for j in hit:   # the candidate at an admissible position, and whatever may trade places with it in the order
        if j >= p0:
            ok.update(tail_pool)
        ok.update(int(i) for i in idx_all[np.abs(zs_all - zs_all[j]) < 2 * tol / T + 1e-7])
    return ok, len(ok) > 1


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


def compare_with_oracle(model, sched, reqs, weights_cpu, tol, *, oracle_dtype=np.float64, plain_too=True,
                        noise_relative=False, **kw):
    """The whole check of one configuration: the oracle in the data path's rounding mode runs free
    (its own tokens fed back); the GPU is teacher-forced with those tokens; traces must be equal word
    for word (sampled tokens apart), logits within the tolerance, tokens by the margin rule.  For the
    bf16 data path the plain high-precision oracle (no rounding hook) runs on the same forced tokens.

    Tolerance.  `tol` is the absolute max-abs bound (2e-2 for bf16, 1e-4 for the fp32 mode).  With
    `noise_relative` (the large layer shapes) the bound is taken from the arithmetic instead: two
    evaluations that are both correct and differ only in where values are rounded to 16 bits (the two
    oracles) differ by max-abs N_max and rms N_rms on these very inputs; an implementation cannot be
    asked to be closer to either of them than they are to each other.  Then the GPU must satisfy
      max|gpu - rounding oracle| <= max(tol, 1.5 N_max), rms(gpu - rounding oracle) <= N_rms,
      max|gpu - plain oracle|    <= max(tol, 1.5 N_max), rms(gpu - plain oracle)  <= 1.25 N_rms
    (the rms bounds are the sharp ones: a maximum over 10^7 to 10^8 entries fluctuates by tens of per
    cent from one realisation of the rounding to the next), and the token rule uses the max bound as
    the logit tolerance."""
    matched_round = O2.round_bf16 if model.dtype == "bf16" else None
    W = O2.Weights(model, weights_as_numpy(model, weights_cpu), dtype=oracle_dtype)
    opol = "pause_resume" if kw.get("policy", B.POLICY_CHUNKED) == B.POLICY_PAUSE_RESUME else "chunked"
    ora = OS.run(model, sched, W, reqs, act_round=matched_round, policy=opol)
    trace, toks, logits, its = gpu_run_forced(model, sched, reqs, weights_cpu, ora["tokens"], **kw)
    assert_traces_equal([{**r, "sampled": []} for r in trace], [{**r, "sampled": []} for r in ora["trace"]])
    lo = np.stack([np.asarray(row, dtype=np.float32) for (_, _, _, _, row) in ora["logits"]])
    assert logits.shape == lo.shape
    lg = logits

    def dist(a, b):   # (max-abs, rms) of a - b, row by row to bound temporary memory
        mx, ss = 0.0, 0.0
        for i in range(a.shape[0]):
            dd = a[i].astype(np.float64) - b[i]
            mx = max(mx, float(np.abs(dd).max()))
            ss += float(np.dot(dd, dd))
        return mx, float(np.sqrt(ss / a.size))

    err, err_rms = dist(lg, lo)
    out = dict(err=err, err_rms=err_rms, err_plain=err, err_plain_rms=err_rms, noise_max=0.0, noise_rms=0.0,
               logit_std=float(lo[: min(64, lo.shape[0])].std()), trace=trace, toks=toks, ora=ora, its=its, logits=logits)
    tol_eff = tol
    if matched_round is not None and (plain_too or noise_relative):
        plain = OS.run(model, sched, W, reqs, act_round=None, forced=ora["tokens"], policy=opol)
        lp = np.stack([np.asarray(row, dtype=np.float32) for (_, _, _, _, row) in plain["logits"]])
        (ep, ep_rms), (nm, n_rms) = dist(lg, lp), dist(lo, lp)
        out.update(err_plain=ep, err_plain_rms=ep_rms, noise_max=nm, noise_rms=n_rms)
        if noise_relative:
            tol_eff = max(tol, 1.5 * out["noise_max"])
            msg = (f"gpu vs rounding oracle max {err:.3e} rms {err_rms:.3e}; gpu vs plain oracle max {out['err_plain']:.3e} "
                   f"rms {out['err_plain_rms']:.3e}; rounding oracle vs plain oracle max {out['noise_max']:.3e} rms {out['noise_rms']:.3e}")
            assert err_rms <= out["noise_rms"], msg
            assert out["err_plain"] <= max(tol, 1.5 * out["noise_max"]), msg
            assert out["err_plain_rms"] <= 1.25 * out["noise_rms"], msg
    out["tol"] = tol_eff
    assert err <= tol_eff, f"max-abs logit error {err:.3e} against the oracle exceeds {tol_eff:.3e}"
    out["n_margin"] = assert_tokens_within_margin(ora, reqs, toks, tol_eff)
    return out
