"""GPU parity of the control plane (scheduler, allocator, ring protocol): the device
trace must equal the oracle's, word for word."""
import numpy as np
import pytest

from oracle import scheduler as O1
from paper_2604_07609_b200 import binding as B
from synth import make_requests, model_cfg, sched_cfg
from synth.workload import Request

from gpu_util import assert_traces_equal, oracle_control_trace, run_control_only

pytestmark = pytest.mark.gpu


def _check(model, sched, reqs, **kw):
    trace, toks, st, its = run_control_only(model, sched, reqs, **kw)
    assert st.device_status == 0
    tr_o, toks_o = oracle_control_trace(sched, reqs, trace, model.vocab)
    assert_traces_equal(trace, tr_o)
    assert toks == toks_o
    assert st.free_blocks == sched.n_blocks and st.reserved_blocks == 0 and st.batch_live == 0
    return trace, st, its


@pytest.mark.parametrize("mode", [B.EXEC_PERSISTENT, B.EXEC_STEPPED, B.EXEC_HOST_GRAPH, B.EXEC_HOST_LAUNCHES],
                         ids=["persistent", "stepped", "host-graph", "host-launches"])
def test_config1_trace_bit_exact(mode):
    model, sched = model_cfg(1), sched_cfg(1)
    trace, st, _ = _check(model, sched, make_requests(1), exec_mode=mode)
    assert trace[0]["W"] == 7 and len(trace[0]["admitted"]) == 8     # all visible to the first iteration


def test_host_driven_arm_with_requests_arriving_while_it_runs():
    """The host-driven comparison arm (a library thread launches one iteration per CUDA graph and waits for it):
    half of the requests arrive after the start; the trace equals the oracle's replay with the logged watermarks."""
    model, sched = model_cfg(1), sched_cfg(1)
    trace, st, _ = _check(model, sched, make_requests(1), exec_mode=B.EXEC_HOST_GRAPH, trickle=4)
    assert st.launches >= len(trace)        # one graph launch per iteration


def test_tiny_pool_head_of_line_blocking():
    model = model_cfg(1)
    sched = sched_cfg(1, n_blocks=9, max_batch=4, prefill_chunk_tokens=24)
    rng = np.random.default_rng(11)
    reqs = [Request(t, 0.0, rng.integers(0, 4096, size=int(p)).astype(np.int32), int(n))
            for t, (p, n) in enumerate([(40, 8), (64, 32), (5, 2), (33, 17), (64, 1), (1, 1), (17, 30)])]
    trace, st, _ = _check(model, sched, reqs)
    assert max(r["reserved"] for r in trace) <= 9


def test_relaunch_with_small_iteration_budget_continues_bit_exactly():
    model, sched = model_cfg(1), sched_cfg(1)
    reqs = make_requests(1)
    full, _, st_full, _ = run_control_only(model, sched, reqs)
    cut, _, st_cut, _ = run_control_only(model, sched, reqs, iteration_budget=7)
    assert st_cut.launches > st_full.launches and st_cut.launches >= len(full) // 7
    assert_traces_equal(cut, full)


def test_slot_reuse_and_backpressure():
    model = model_cfg(1)
    sched = sched_cfg(1, n_slots=4, max_batch=2)
    rng = np.random.default_rng(5)
    eng = B.Blink(model, sched, control_only=True, trace_words=1 << 20, idle_exit_us=300_000)
    try:
        mk = lambda: rng.integers(0, 4096, size=20).astype(np.int32)
        for i in range(4):
            assert eng.blink_submit(mk(), 6) == i
        assert eng.blink_submit(mk(), 6, raise_on_error=False) == B.BLINK_EAGAIN     # ring full
        ev = eng.drain(24, timeout_s=30)
        assert sorted(set(int(t) for t in ev["ticket"])) == [0, 1, 2, 3]
        for i in range(4, 8):                                                         # slots were recycled
            assert eng.blink_submit(mk(), 3) == i
        ev2 = eng.drain(12, timeout_s=30)
        assert sorted(set(int(t) for t in ev2["ticket"])) == [4, 5, 6, 7]
        for t in range(4, 8):
            idx = [int(e["index"]) for e in ev2 if e["ticket"] == t]
            assert idx == [0, 1, 2]
        # argument checks
        assert eng.blink_submit(np.zeros(65, np.int32), 3, raise_on_error=False) == B.BLINK_EINVAL
        assert eng.blink_submit(np.array([4096], np.int32), 3, raise_on_error=False) == B.BLINK_EINVAL
        assert eng.blink_submit(mk(), 0, raise_on_error=False) == B.BLINK_EINVAL
        assert eng.blink_submit(mk(), 3, top_k=65, raise_on_error=False) == B.BLINK_EINVAL
    finally:
        assert eng.blink_destroy() == B.BLINK_OK


def test_idle_exit_and_relaunch_on_submit():
    import time
    model, sched = model_cfg(1), sched_cfg(1)
    eng = B.Blink(model, sched, control_only=True, idle_exit_us=50_000)
    try:
        time.sleep(0.5)
        assert eng.blink_get_stats().loop_state == B.LOOP_EXIT_IDLE       # left the GPU on its own
        eng.blink_submit(np.arange(10, dtype=np.int32), 4)
        ev = eng.drain(4, timeout_s=30)
        assert len(ev) == 4 and eng.blink_get_stats().launches == 2
        assert eng.blink_stop(final=True) == B.BLINK_OK
        assert eng.blink_submit(np.arange(10, dtype=np.int32), 4, raise_on_error=False) == B.BLINK_ESTOPPED
    finally:
        assert eng.blink_destroy() == B.BLINK_OK


def test_config3_and_config5_streams_trace_at_full_scale():
    """Traces do not depend on the model math (fixed output lengths), so the full request
    streams of the 8B and MoE configurations are checked in control-only mode."""
    for cfg_i, n_blocks in ((3, 60000), (5, 60000)):
        model = model_cfg(cfg_i)
        sched = sched_cfg(cfg_i, n_blocks=n_blocks)
        reqs = make_requests(cfg_i)
        trace, st, its = _check(model, sched, reqs, trace_words=1 << 27)
        assert sum(len(r["sampled"]) for r in trace) == sum(r.max_new for r in reqs)
        assert max(len(r["scheduled"]) for r in trace) <= 256
        dt = (its["t_end_ns"] - its["t_begin_ns"]).astype(np.float64)
        print(f"config {cfg_i}: {len(trace)} iterations, control plane median {np.median(dt) / 1e3:.1f} us/iter")


def test_timestamps_and_event_order():
    model, sched = model_cfg(1), sched_cfg(1)
    reqs = make_requests(1)
    eng = B.Blink(model, sched, control_only=True, idle_exit_us=300_000)
    try:
        for r in reqs:
            eng.submit_request(r)
        ev = eng.drain(8 * 32, timeout_s=30)
        off = eng.blink_get_stats().device_clock_offset_ns
        for t in range(8):
            e = np.sort(ev[ev["ticket"] == t], order="index")
            assert list(e["index"]) == list(range(32))
            assert e["is_first"][0] == 1 and e["is_last"][-1] == 1 and e["is_last"][:-1].sum() == 0
            assert np.all(np.diff(e["t_device_ns"].astype(np.int64)) > 0)
            ttft_ns = int(e["t_device_ns"][0]) + off - int(e["t_submit_ns"][0])
            assert -1_000_000 < ttft_ns < 2_000_000_000
    finally:
        assert eng.blink_destroy() == B.BLINK_OK


def test_eos_retires_a_request_early_and_frees_its_blocks():
    """A request whose eos_id is a token it emits before max_new: it is retired in that iteration
    (blocks pushed back, reservation released, finished flag in the published count) and the trace
    equals the oracle's, which is given the same eos ids."""
    model = model_cfg(1)
    sched = sched_cfg(1, max_batch=4, n_blocks=64)
    reqs = make_requests(1)
    # control-only tokens are a fixed function of (ticket, index): pick, for every other request, the
    # token it will emit at index 5 (unless it shows up earlier, then that earlier index ends it)
    for r in reqs[::2]:
        r.eos_id = O1.fake_token(r.ticket, 5, model.vocab)
    eng = B.Blink(model, sched, control_only=True, start_paused=True, trace_words=1 << 20, idle_exit_us=300_000)
    try:
        for r in reqs:
            eng.submit_request(r)
        eng.blink_start()
        tr_o, toks_o, _ = O1.simulate([O1.SimRequest(r.ticket, r.n_prompt, r.max_new, r.eos_id, r.prompt) for r in reqs],
                                      sched.max_batch, sched.prefill_chunk_tokens, sched.n_blocks, sched.block_size,
                                      vocab=model.vocab)
        total = sum(len(v) for v in toks_o.values())
        assert total < sum(r.max_new for r in reqs)                  # some requests really ended early
        ev = eng.drain(total, timeout_s=60)
        eng.blink_stop(final=False)
        st = eng.blink_get_stats()
        trace = B.parse_trace(eng.blink_get_trace())
    finally:
        assert eng.blink_destroy() == B.BLINK_OK
    assert st.device_status == 0
    assert_traces_equal(trace, tr_o)
    assert B.tokens_by_ticket(ev) == toks_o
    assert st.free_blocks == sched.n_blocks and st.reserved_blocks == 0 and st.batch_live == 0
    for r in reqs:
        e = np.sort(ev[ev["ticket"] == r.ticket], order="index")
        assert len(e) == len(toks_o[r.ticket])
        assert e["is_last"][-1] == 1 and e["is_last"][:-1].sum() == 0
        if r.eos_id >= 0:
            assert len(e) <= 6 and int(e["token"][-1]) == r.eos_id


def test_a_wait_that_runs_out_unwinds_the_loop_with_a_status():
    """Every wait inside the kernel is bounded.  Here the bound (5 ms) is set below the idle-exit time
    (1 s): once the queue is empty the control plane keeps polling it while the other CTAs of the grid
    wait at the grid barrier for the next step, and nothing ends that wait in time.  The waiting CTAs
    must record the time-out, every CTA must leave the GPU, the host calls must report the device
    error, and the context must still be destroyed cleanly (no trap, no hang: the CUDA context stays
    usable, which the tests that run after this one rely on)."""
    import time
    import torch
    from synth import make_weights
    model, sched = model_cfg(1, dtype="fp32"), sched_cfg(1)
    w = make_weights(model, 1, "cpu").cuda()
    kv = torch.zeros(sched.n_blocks * B.kv_bytes_per_block(model, sched.block_size), dtype=torch.uint8, device="cuda")
    eng = B.Blink(model, sched, w, kv, idle_exit_us=1_000_000, wait_limit_ms=5)
    try:
        rng = np.random.default_rng(3)
        eng.blink_submit(rng.integers(0, model.vocab, size=20).astype(np.int32), 4)
        ev = eng.drain(4, timeout_s=30)            # real work completes: the limit is far above a step's time
        assert len(ev) == 4
        t0 = time.monotonic()
        while eng.blink_get_stats().loop_state == B.LOOP_RUNNING and time.monotonic() - t0 < 5:
            time.sleep(0.01)
        st = eng.blink_get_stats()
        assert st.loop_state == B.LOOP_EXIT_ERROR, st.loop_state
        assert st.device_status == 1                 # the grid-barrier wait ran out
        assert time.monotonic() - t0 < 0.9           # long before the idle exit: it was the wait limit
        with pytest.raises(B.BlinkError) as e:
            eng.blink_poll(16, 1000)
        assert e.value.code == B.BLINK_EDEVICE
        assert eng.blink_submit(np.arange(8, dtype=np.int32), 2, raise_on_error=False) == B.BLINK_EDEVICE
    finally:
        assert eng.blink_destroy() == B.BLINK_OK
    # the CUDA context is intact: a fresh loop on the same device works
    trace, toks, st2, _ = run_control_only(model_cfg(1), sched_cfg(1), make_requests(1))
    assert st2.device_status == 0 and len(toks) == 8


def test_pause_resume_policy_trace_bit_exact():
    """The paper's own inline prefill (whole prompts in prefill-only steps while decoding is paused for one
    step): device trace equal to the oracle's under the same policy, with requests that arrive while the
    loop is running (the logged watermarks are replayed)."""
    model = model_cfg(1)
    sched = sched_cfg(1, max_batch=6, prefill_chunk_tokens=160, n_blocks=128, max_prompt=64, max_new=32)
    rng = np.random.default_rng(17)
    reqs = [Request(t, 0.0, rng.integers(0, 4096, size=int(p)).astype(np.int32), int(n))
            for t, (p, n) in enumerate(zip(rng.integers(5, 65, size=40), rng.integers(1, 33, size=40)))]
    trace, toks, st, _ = run_control_only(model, sched, reqs, policy=B.POLICY_PAUSE_RESUME, trickle=30)
    assert st.device_status == 0
    tr_o, toks_o = oracle_control_trace(sched, reqs, trace, model.vocab, policy="pause_resume")
    assert_traces_equal(trace, tr_o)
    assert toks == toks_o
    kinds = [{s[2] for s in r["scheduled"]} for r in trace]
    assert all(len(k) == 1 for k in kinds) and {1} in kinds and {2} in kinds      # never a mixed step
    assert all(s[3] == 0 and s[4] == reqs[s[1]].n_prompt for r in trace for s in r["scheduled"] if s[2] == 1)
    assert st.free_blocks == sched.n_blocks and st.reserved_blocks == 0 and st.batch_live == 0
    # a prefill budget below the longest accepted prompt cannot run whole prompts: refused at create
    with pytest.raises(B.BlinkError):
        B.Blink(model, sched_cfg(1, prefill_chunk_tokens=32, max_prompt=64), control_only=True, policy=B.POLICY_PAUSE_RESUME)


def test_cancel_retires_a_running_request_and_the_trace_equals_the_oracles():
    """blink_cancel on a request that is generating: the device retires it at a step boundary (blocks and
    reservation returned, batch slot released), its tokens so far are delivered, one closing event follows,
    and the trace equals the oracle's when the oracle is told in which iteration the mark was seen."""
    import time
    model = model_cfg(1)
    sched = sched_cfg(1, max_batch=3, n_blocks=2048, max_prompt=64, max_new=30000, n_slots=16)
    rng = np.random.default_rng(23)
    mk = lambda n: rng.integers(0, 4096, size=n).astype(np.int32)
    reqs = [Request(0, 0.0, mk(40), 12), Request(1, 0.0, mk(25), 30000), Request(2, 0.0, mk(33), 20),
            Request(3, 0.0, mk(10), 15), Request(4, 0.0, mk(50), 9)]
    eng = B.Blink(model, sched, control_only=True, start_paused=True, trace_words=1 << 24, idle_exit_us=300_000)
    try:
        for r in reqs:
            eng.submit_request(r)
        eng.blink_start()
        evs, closing = [], None
        t0 = time.monotonic()
        asked = False
        while closing is None and time.monotonic() - t0 < 30:
            e = eng.blink_poll(4096, 1000)
            if len(e):
                evs.append(e)
                if not asked and (e["ticket"] == 1).sum() > 0:
                    assert eng.blink_cancel(1) == B.BLINK_OK       # ticket 1 is generating: stop it
                    asked = True
                c = e[(e["ticket"] == 1) & (e["is_last"] == 1)]
                if len(c):
                    closing = c[0]
        assert closing is not None and int(closing["token"]) == -1
        # everything else runs to its end
        rest = sum(r.max_new for r in reqs if r.ticket != 1)
        got = sum(int((e["ticket"] != 1).sum()) for e in evs)
        while got < rest and time.monotonic() - t0 < 60:
            e = eng.blink_poll(4096, 1000)
            evs.append(e)
            got += int((e["ticket"] != 1).sum())
        assert got == rest
        assert eng.blink_cancel(1) == B.BLINK_EINVAL              # gone
        assert eng.blink_cancel(99) == B.BLINK_EINVAL             # never existed
        eng.blink_stop(final=False)
        st = eng.blink_get_stats()
        trace = B.parse_trace(eng.blink_get_trace())
    finally:
        assert eng.blink_destroy() == B.BLINK_OK
    assert st.device_status == 0
    ev = np.concatenate(evs)
    mine = np.sort(ev[(ev["ticket"] == 1) & (ev["token"] >= 0)], order="index")
    n1 = len(mine)
    assert 0 < n1 < 30000 and list(mine["index"]) == list(range(n1)) and mine["is_last"].sum() == 0
    assert int(closing["index"]) == n1
    it_c = next(i for i, r in enumerate(trace) if 1 in r["finished"])
    tr_o, toks_o, _ = O1.simulate([O1.SimRequest(r.ticket, r.n_prompt, r.max_new, r.eos_id, r.prompt) for r in reqs],
                                  sched.max_batch, sched.prefill_chunk_tokens, sched.n_blocks, sched.block_size,
                                  watermarks=[r["W"] for r in trace], vocab=model.vocab, cancels={it_c: [1]})
    assert_traces_equal(trace, tr_o)
    assert len(toks_o[1]) == n1 and [int(t) for t in mine["token"]] == toks_o[1]
    assert st.free_blocks == sched.n_blocks and st.reserved_blocks == 0 and st.batch_live == 0
