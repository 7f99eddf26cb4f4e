"""GPU parity of the whole step (forward + sampling) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import sampler as S
from oracle import transformer as O2
from paper_2604_07609_b200 import binding as B
from synth import make_requests, make_weights, model_cfg, sched_cfg

from gpu_util import assert_tokens_within_margin, assert_traces_equal, compare_with_oracle, gpu_run_forced, oracle_run

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4     # max-abs logit error, fp32 reference mode
TOL_BF16 = 2e-2     # max-abs logit error, bf16 mode


def _compare(model, sched, reqs, weights, act_round, tol, **kw):
    """Oracle (in the data path's rounding mode) vs GPU under teacher forcing: traces, logits within
    `tol`, tokens by the margin rule; for bf16 also the error against the plain high-precision oracle,
    which must meet the same tolerance."""
    r = compare_with_oracle(model, sched, reqs, weights, tol, **kw)
    if model.dtype == "bf16":
        print(f"  max-abs logit error: {r['err']:.3e} against the oracle rounding where the data path stores 16-bit "
              f"values, {r['err_plain']:.3e} against the plain high-precision oracle (the two oracles differ by "
              f"{r['noise_max']:.3e})")
        assert r["err_plain"] <= tol, r["err_plain"]
    return r["err"], r["n_margin"], r["trace"], r["toks"], r["ora"]


def test_config1_fp32_reference_mode_logits_tokens_trace():
    model, sched = model_cfg(1, dtype="fp32"), sched_cfg(1)
    reqs = make_requests(1)
    w = make_weights(model, 1234, "cpu")
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, None, TOL_FP32)
    print(f"C1 fp32: max-abs logit error {err:.3e}, {n_margin} in-margin decisions")
    assert err <= TOL_FP32
    assert toks == ora["tokens"]           # unconditional bit-exact token gate of the small configuration
    assert_traces_equal(trace, ora["trace"])


def test_config1_bf16_logits_within_tolerance():
    model, sched = model_cfg(1, dtype="bf16"), sched_cfg(1)
    reqs = make_requests(1)
    w = make_weights(model, 1234, "cpu")
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16)
    print(f"C1 bf16: max-abs logit error {err:.3e}, {n_margin} in-margin decisions")
    assert err <= TOL_BF16


def test_stepped_mode_matches_persistent_mode_bitwise():
    model, sched = model_cfg(1, dtype="fp32"), sched_cfg(1)
    reqs = make_requests(1, n_requests=4)
    w = make_weights(model, 99, "cpu", random_gains=True)
    a = gpu_run_forced(model, sched, reqs, w, None, exec_mode=B.EXEC_PERSISTENT)
    b = gpu_run_forced(model, sched, reqs, w, None, exec_mode=B.EXEC_STEPPED)
    assert a[1] == b[1]
    assert np.array_equal(a[2], b[2])
    assert_traces_equal(a[0], b[0])


@pytest.mark.parametrize("mode", [B.EXEC_HOST_GRAPH, B.EXEC_HOST_LAUNCHES], ids=["graph-per-iteration", "launch-per-phase"])
def test_host_driven_arms_match_persistent_mode_bitwise(mode):
    """The comparison arms (a host thread launches one iteration at a time and waits for it) run the same
    device code: same trace, same tokens, same logits bit for bit; blink_step is refused there."""
    model, sched = model_cfg(1, dtype="fp32"), sched_cfg(1)
    reqs = make_requests(1, n_requests=4)
    w = make_weights(model, 99, "cpu", random_gains=True)
    a = gpu_run_forced(model, sched, reqs, w, None, exec_mode=B.EXEC_PERSISTENT)
    b = gpu_run_forced(model, sched, reqs, w, None, exec_mode=mode)
    assert a[1] == b[1]
    assert np.array_equal(a[2], b[2])
    assert_traces_equal(a[0], b[0])


def test_gqa_random_gains_chunked_prefill_small_chunk():
    """Grouped-query heads (4 q per kv head), head_dim 128, non-unit norm gains, and a chunk
    budget smaller than the prompts so prefill spans several iterations and mixes with decode."""
    model = model_cfg(1, n_q_heads=4, n_kv_heads=1, head_dim=128, d_model=256, dtype="fp32")
    sched = sched_cfg(1, prefill_chunk_tokens=24, max_batch=4, n_blocks=64)
    reqs = make_requests(1, n_requests=6)
    w = make_weights(model, 7, "cpu", random_gains=True)
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, None, TOL_FP32)
    print(f"GQA fp32: max-abs logit error {err:.3e}")
    assert err <= TOL_FP32
    assert any(s[2] == 1 for r in trace for s in r["scheduled"]) and any(
        {1, 2} <= {s[2] for s in r["scheduled"]} for r in trace)


def test_topk_sampling_end_to_end_fp32():
    model, sched = model_cfg(1, dtype="fp32"), sched_cfg(1)
    reqs = make_requests(1, n_requests=4)
    for r in reqs:
        r.top_k, r.temperature = 50, 0.8
    w = make_weights(model, 5, "cpu")
    # the draw is identical on both sides: tokens are the oracle's except where a candidate-set or
    # inverse-CDF boundary lies inside the logit tolerance (checked by the margin rule in _compare)
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, None, TOL_FP32)
    agree = sum(toks[t][i] == ora["sampled"][t][i] for t in toks for i in range(len(toks[t])))
    total = sum(len(v) for v in toks.values())
    print(f"top-k end to end: {agree}/{total} tokens identical, {n_margin} decisions inside the margin")
    assert total - agree <= n_margin


def test_sampler_alone_bit_exact_on_oracle_logits():
    rng = np.random.default_rng(3)
    V, rows = 128256, 48
    logits = (rng.normal(size=(rows, V)) * 1.3).astype(np.float32)
    logits[0, :] = 0.0                              # all equal: ties must break to the lowest indices
    logits[1, 1000:1200] = logits[1].max() + 1.0    # a plateau larger than k
    logits[2] = np.round(logits[2] * 2) / 2         # heavy quantisation: many exact ties
    top_k = np.array([0 if i % 3 == 0 else (50 if i % 3 == 1 else 7) for i in range(rows)], dtype=np.int32)
    top_k[:3] = [50, 50, 64]
    temp = np.where(np.arange(rows) % 2 == 0, 0.8, 1.3).astype(np.float32)
    ticket = np.arange(rows, dtype=np.uint64) * 977 + (1 << 33)
    gen = (np.arange(rows) * 5 % 97).astype(np.int32)
    seed = (np.arange(rows, dtype=np.uint64) * 0x9E3779B97F4A7C15) ^ np.uint64(0xB11C0003)
    got = B.blink_sample(torch.from_numpy(logits).cuda(), top_k, temp, ticket, gen, seed)
    for r in range(rows):
        want = S.sample(logits[r], int(top_k[r]), float(temp[r]), int(ticket[r]), int(gen[r]), int(seed[r]))
        assert int(got[r]) == want, (r, int(got[r]), want)
    # many draws on one row: the empirical distribution is the oracle's
    row = logits[5:6].repeat(400, axis=0)
    n = 400
    g2 = B.blink_sample(torch.from_numpy(row).cuda(), np.full(n, 50, np.int32), np.full(n, 0.8, np.float32),
                        np.full(n, 7, np.uint64), np.arange(n, dtype=np.int32), np.full(n, 42, np.uint64))
    w2 = [S.sample(logits[5], 50, 0.8, 7, i, 42) for i in range(n)]
    assert list(g2) == w2


# ---- tensor-core (tcgen05 / TMEM / TMA) path of the dense contractions ---------------------------
@pytest.mark.parametrize("fusion", [B.FUSION_OFF, B.FUSION_ON], ids=["separate-phases", "fused-epilogues"])
def test_config1_bf16_tensor_core_path_matches_oracle(fusion):
    model, sched = model_cfg(1, dtype="bf16"), sched_cfg(1)
    reqs = make_requests(1)
    w = make_weights(model, 1234, "cpu")
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16, gemm_impl=B.GEMM_TC,
                                               epilogue_fusion=fusion)
    print(f"C1 bf16 tensor cores: max-abs logit error {err:.3e}, {n_margin} in-margin decisions")
    assert err <= TOL_BF16


@pytest.mark.parametrize("gemm,fusion", [(B.GEMM_TC, B.FUSION_ON), (B.GEMM_TC, B.FUSION_OFF), (B.GEMM_TC_PAIR, B.FUSION_OFF)],
                         ids=["single-cta-fused", "single-cta", "cta-pairs"])
def test_tensor_core_path_multi_pass_ragged_shapes(gemm, fusion):
    """More than 256 rows in a step (two token passes), 24 k-blocks, 35 n-tiles (an odd number: the
    last CTA pair has one real weight tile), GQA 4:1 with head_dim 128, non-unit gains: every stream-K
    segment kind (whole tile, head, tail) occurs."""
    model = model_cfg(1, d_model=512, n_q_heads=4, n_kv_heads=1, head_dim=128, d_ff=1536, vocab=4480, dtype="bf16")
    sched = sched_cfg(1, prefill_chunk_tokens=300, max_batch=8, n_blocks=256, max_prompt=320, max_new=8)
    rng = np.random.default_rng(21)
    from synth.workload import Request
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 6)
            for t, p in enumerate([310, 17, 301, 64, 129, 256, 5, 300, 33])]
    w = make_weights(model, 77, "cpu", random_gains=True)
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16, gemm_impl=gemm,
                                               epilogue_fusion=fusion)
    print(f"multi-pass tensor cores: max-abs logit error {err:.3e}; max rows/step "
          f"{max(sum(s[4] for s in r['scheduled']) for r in trace)}")
    assert err <= TOL_BF16
    assert max(sum(s[4] for s in r["scheduled"]) for r in trace) > 256


def test_tensor_core_and_cuda_core_paths_agree():
    model, sched = model_cfg(1, dtype="bf16"), sched_cfg(1)
    reqs = make_requests(1, n_requests=4)
    w = make_weights(model, 3, "cpu", random_gains=True)
    forced = {r.ticket: [int(x) for x in np.random.default_rng(r.ticket).integers(0, 4096, size=r.max_new)] for r in reqs}
    a = gpu_run_forced(model, sched, reqs, w, forced, gemm_impl=B.GEMM_SIMT)
    b = gpu_run_forced(model, sched, reqs, w, forced, gemm_impl=B.GEMM_TC, exec_mode=B.EXEC_STEPPED)
    assert np.abs(a[2] - b[2]).max() < TOL_BF16  # same bf16 products, other summation order, so roundings flip
    assert_traces_equal([{**r, "sampled": []} for r in a[0]], [{**r, "sampled": []} for r in b[0]])


@pytest.mark.parametrize("gemm", [B.GEMM_TC, B.GEMM_TC_PAIR], ids=["single-cta", "cta-pairs"])
def test_streaming_weight_layout_round_trip_and_parity(gemm):
    """The GEMM matrices converted in place to the tile-contiguous streaming layout: converting back
    restores every byte, and the loop reading the streaming layout meets the same tolerance."""
    model = model_cfg(1, d_model=512, n_q_heads=4, n_kv_heads=1, head_dim=128, d_ff=1536, vocab=4480, dtype="bf16")
    sched = sched_cfg(1, prefill_chunk_tokens=300, max_batch=8, n_blocks=256, max_prompt=320, max_new=8)
    rng = np.random.default_rng(22)
    from synth.workload import Request
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 6)
            for t, p in enumerate([310, 17, 301, 64, 129, 5])]
    w = make_weights(model, 78, "cpu", random_gains=True)
    wd = w.cuda()
    B.blink_convert_weights(model, wd, B.WEIGHTS_ROW_MAJOR, B.WEIGHTS_STREAMING)
    assert not torch.equal(wd.cpu(), w)
    back = wd.clone()
    B.blink_convert_weights(model, back, B.WEIGHTS_STREAMING, B.WEIGHTS_ROW_MAJOR)
    assert torch.equal(back.cpu(), w)
    # a 128 x 64 tile of wqkv holds exactly the values of the row-major block it came from
    off = B.blink_weight_offset(model, 1)
    K = model.d_model
    tile = wd[off:off + 16384].cpu().view(torch.bfloat16).view(128, 8, 8)          # [row][chunk position][8]
    rm = w[off:off + 128 * K * 2].view(torch.bfloat16).view(128, K)[:, :64].reshape(128, 8, 8)
    for r in (0, 1, 7, 8, 77, 127):
        for c8 in range(8):
            assert torch.equal(tile[r, c8 ^ (r & 7)], rm[r, c8])
    # gate/up: stored row 2 f is gate row f, stored row 2 f + 1 is up row f
    off3, F = B.blink_weight_offset(model, 3), model.d_ff
    tile = wd[off3:off3 + 16384].cpu().view(torch.bfloat16).view(128, 8, 8)
    rm3 = w[off3:off3 + 2 * F * K * 2].view(torch.bfloat16).view(2 * F, K)
    for r in (0, 1, 2, 9, 126, 127):
        src = rm3[(r & 1) * F + (r >> 1), :64].reshape(8, 8)
        for c8 in range(8):
            assert torch.equal(tile[r, c8 ^ (r & 7)], src[c8])
    err, _, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16, gemm_impl=gemm,
                                        weights_layout=B.WEIGHTS_STREAMING)
    print(f"streaming layout: max-abs logit error {err:.3e}")
    # the SIMT path cannot read the streaming layout: refused, not misread
    with pytest.raises(B.BlinkError):
        gpu_run_forced(model, sched, reqs, w, ora["tokens"], gemm_impl=B.GEMM_SIMT, weights_layout=B.WEIGHTS_STREAMING)


@pytest.mark.parametrize("dtype,tol,kw", [("fp32", TOL_FP32, {}),
                                           ("bf16", TOL_BF16, dict(gemm_impl=B.GEMM_TC, weights_layout=B.WEIGHTS_STREAMING))],
                         ids=["fp32-simt", "bf16-tensor-cores-streaming"])
def test_routed_experts_match_oracle(dtype, tol, kw):
    """Top-2 of 4 experts: router on the fp32 normed rows, stable grouping by expert, per-expert
    GEMMs on gathered rows, gate-weighted sum into the residual stream."""
    model = model_cfg(1, n_experts=4, top_k_experts=2, d_ff=512, dtype=dtype)
    sched = sched_cfg(1, prefill_chunk_tokens=40, max_batch=6, n_blocks=128)
    reqs = make_requests(1, n_requests=6)
    for r in reqs:
        r.max_new = 8
    w = make_weights(model, 31, "cpu", random_gains=True)
    err, _, trace, toks, ora = _compare(model, sched, reqs, w, None, tol, **kw)
    print(f"routed experts {dtype}: max-abs logit error {err:.3e}")


def test_decode_attention_many_rows_whole_and_split_units():
    """64 requests with contexts of a few hundred tokens: the flat (row, kv head, block) tile sequence
    is longer than the number of warps, so sub-ranges hold several tiles and units are both
    handled whole and cut (partial records merged); prefill chunks span several requests."""
    model = model_cfg(1, dtype="bf16")
    sched = sched_cfg(1, prefill_chunk_tokens=512, max_batch=64, n_blocks=2048, max_prompt=400, max_new=6, n_slots=128)
    rng = np.random.default_rng(5)
    from synth.workload import Request
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 6)
            for t, p in enumerate(rng.integers(150, 400, size=64))]
    w = make_weights(model, 11, "cpu", random_gains=True)
    err, _, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16)
    print(f"64 rows, long contexts: max-abs logit error {err:.3e}; rows/step up to "
          f"{max(sum(s[4] for s in r['scheduled']) for r in trace)}")


def test_decode_attention_few_long_rows():
    """Two requests with contexts of 1200 and 1900 tokens: fewer tiles than warps, so every (row, kv head)
    unit is cut into sub-ranges of the minimum size and merged from more than ten partial records."""
    model = model_cfg(1, dtype="bf16")
    sched = sched_cfg(1, prefill_chunk_tokens=512, max_batch=8, n_blocks=512, max_prompt=2048, max_new=6)
    rng = np.random.default_rng(9)
    from synth.workload import Request
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 5)
            for t, p in enumerate([1900, 1200])]
    w = make_weights(model, 12, "cpu", random_gains=True)
    err, _, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16)
    print(f"2 rows, contexts 1200 and 1900: max-abs logit error {err:.3e}")
    assert err <= TOL_BF16


@pytest.mark.parametrize("gemm", [B.GEMM_TC, B.GEMM_TC_PAIR], ids=["single-cta", "cta-pairs"])
def test_gate_up_epilogue_writes_activations_three_ragged_passes(gemm):
    """Streaming layout, more than 512 rows in a step: three token passes, the last one ragged.  The
    gate/up GEMM writes silu(gate) * up itself for the (pass, tile) units whose K it covers in one segment
    and adds partial sums for the others; the SwiGLU phase takes exactly the others."""
    model = model_cfg(1, d_model=512, n_q_heads=4, n_kv_heads=1, head_dim=128, d_ff=1536, vocab=4480, dtype="bf16")
    sched = sched_cfg(1, prefill_chunk_tokens=600, max_batch=8, n_blocks=512, max_prompt=640, max_new=8)
    rng = np.random.default_rng(23)
    from synth.workload import Request
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 5)
            for t, p in enumerate([610, 33, 580, 300, 7])]
    w = make_weights(model, 79, "cpu", random_gains=True)
    err, _, trace, toks, ora = _compare(model, sched, reqs, w, O2.round_bf16, TOL_BF16, gemm_impl=gemm,
                                        weights_layout=B.WEIGHTS_STREAMING)
    rows = max(sum(s[4] for s in r["scheduled"]) for r in trace)
    print(f"three passes, streaming layout: max-abs logit error {err:.3e}; max rows/step {rows}")
    assert err <= TOL_BF16 and rows > 512


# ---- top-p (nucleus) sampling ------------------------------------------------------------------------
def test_top_p_sampler_alone_bit_exact_on_oracle_logits():
    """The nucleus sampler on given logits must pick the oracle's token, row for row: whole-vocabulary
    nuclei of very different sizes (from one token to most of a 128256-entry row), nuclei cut from the
    top-k candidates, rows made of one repeated value or a few values (thousands of exact ties, resolved
    by index), and many draws on one row."""
    rng = np.random.default_rng(9)
    V, rows = 128256, 40
    logits = (rng.normal(size=(rows, V)) * 1.3).astype(np.float32)
    logits[0, :] = 0.25                                  # one value: the order is the index order
    logits[1] = np.round(logits[1])                      # about ten distinct values, tens of thousands of ties each
    logits[2, 777] = 40.0                                # one dominant token: the nucleus is that token
    logits[3] = np.round(logits[3] * 4) / 4
    top_k = np.array([0, 0, 0, 0] + [(0, 50, 0, 64, 7)[i % 5] for i in range(rows - 4)], dtype=np.int32)
    top_p = np.array([0.9, 0.5, 0.9, 0.7] + [(0.9, 0.8, 0.3, 0.95, 0.5, 0.999, 0.05)[i % 7] for i in range(rows - 4)], dtype=np.float32)
    temp = np.where(np.arange(rows) % 2 == 0, 0.8, 1.3).astype(np.float32)
    ticket = np.arange(rows, dtype=np.uint64) * 613 + (1 << 34)
    gen = (np.arange(rows) * 7 % 89).astype(np.int32)
    seed = (np.arange(rows, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15)) ^ np.uint64(0xB11C0009)
    dev = torch.from_numpy(logits).cuda()
    got = B.blink_sample_top_p(dev, top_k, temp, top_p, ticket, gen, seed)
    for r in range(rows):
        want = S.sample(logits[r], int(top_k[r]), float(temp[r]), int(ticket[r]), int(gen[r]), int(seed[r]), float(top_p[r]))
        assert int(got[r]) == want, (r, int(got[r]), want, int(top_k[r]), float(top_p[r]))
    # top_p outside (0, 1) switches the cut off: same tokens as the plain entry point
    off = np.where(np.arange(rows) % 2 == 0, 0.0, 1.0).astype(np.float32)
    assert np.array_equal(B.blink_sample_top_p(dev, top_k, temp, off, ticket, gen, seed),
                          B.blink_sample(dev, top_k, temp, ticket, gen, seed))
    # many draws on two rows (a continuous one and the all-equal one)
    n = 120
    for r, p in ((5, 0.9), (0, 0.6), (1, 0.8)):
        rowdev = dev[r:r + 1].repeat(n, 1).contiguous()
        g2 = B.blink_sample_top_p(rowdev, np.zeros(n, np.int32), np.full(n, 0.8, np.float32), np.full(n, p, np.float32),
                                  np.full(n, 11, np.uint64), np.arange(n, dtype=np.int32), np.full(n, 4242, np.uint64))
        idx, q = S.nucleus(logits[r], 0, 0.8, p)
        qs, M = np.cumsum(np.array(q, dtype=object)), sum(q)
        for i in range(n):
            x24 = S.philox_word(11, i, 4242) >> 8
            target = (x24 * M) >> 24
            j = int(np.argmax(qs > target))
            assert int(g2[i]) == int(idx[j]), (r, p, i)


def test_top_p_sampling_end_to_end_fp32():
    model, sched = model_cfg(1, dtype="fp32"), sched_cfg(1)
    reqs = make_requests(1, n_requests=6)
    for i, r in enumerate(reqs):
        r.temperature, r.top_p = 0.8, (0.9, 0.6)[i % 2]
        r.top_k = 0 if i < 4 else 20
    w = make_weights(model, 6, "cpu")
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, None, TOL_FP32)
    agree = sum(toks[t][i] == ora["sampled"][t][i] for t in toks for i in range(len(toks[t])))
    total = sum(len(v) for v in toks.values())
    print(f"top-p end to end: {agree}/{total} tokens identical, {n_margin} decisions inside the margin")
    assert total - agree <= n_margin


def test_pause_resume_policy_logits_and_tokens_fp32():
    """Whole-prompt prefill steps of several requests at once, decode paused meanwhile: same model math."""
    model = model_cfg(1, dtype="fp32")
    sched = sched_cfg(1, max_batch=4, prefill_chunk_tokens=128, n_blocks=64)
    reqs = make_requests(1, n_requests=7)
    for r in reqs:
        r.max_new = 9
    w = make_weights(model, 8, "cpu", random_gains=True)
    err, n_margin, trace, toks, ora = _compare(model, sched, reqs, w, None, TOL_FP32, policy=B.POLICY_PAUSE_RESUME)
    print(f"pause-and-resume fp32: max-abs logit error {err:.3e}")
    assert all(len({s[2] for s in r["scheduled"]}) == 1 for r in trace)
    assert any(len(r["scheduled"]) > 1 and r["scheduled"][0][2] == 1 for r in trace)     # several prompts in one step


def test_bf16_stepped_and_persistent_modes_agree_on_the_tensor_core_path():
    """The persistent loop reads, through TMA, buffers that earlier phases of the same kernel wrote with
    ordinary stores (normed rows, K/V rows, attention output, SwiGLU output); the stepped mode has a kernel
    boundary between any two phases.  Both must give the same trace, logits within the bf16 tolerance of
    each other and of the oracle, and tokens by the margin rule (split-K sums land in arrival order, so
    the two are not bit-identical)."""
    model = model_cfg(1, d_model=512, n_q_heads=4, n_kv_heads=1, head_dim=128, d_ff=1536, vocab=4480, dtype="bf16")
    sched = sched_cfg(1, prefill_chunk_tokens=300, max_batch=8, n_blocks=256, max_prompt=320, max_new=8)
    rng = np.random.default_rng(24)
    from synth.workload import Request
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 8)
            for t, p in enumerate([300, 40, 129, 257, 16, 310])]
    w = make_weights(model, 79, "cpu", random_gains=True)
    runs = {}
    for name, mode in (("persistent", B.EXEC_PERSISTENT), ("stepped", B.EXEC_STEPPED)):
        runs[name] = compare_with_oracle(model, sched, reqs, w, TOL_BF16, gemm_impl=B.GEMM_AUTO,
                                         weights_layout=B.WEIGHTS_STREAMING, exec_mode=mode)
        assert runs[name]["err_plain"] <= TOL_BF16
    a, b = runs["persistent"], runs["stepped"]
    assert_traces_equal([{**r, "sampled": []} for r in a["trace"]], [{**r, "sampled": []} for r in b["trace"]])
    d = float(np.abs(a["logits"] - b["logits"]).max())
    print(f"bf16 persistent vs stepped: max-abs logit difference {d:.3e} (vs oracle {a['err']:.3e} / {b['err']:.3e})")
    assert d <= TOL_BF16
