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
