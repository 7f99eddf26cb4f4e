"""GPU parity at the layer shapes that are benchmarked (the kernel instances, tile counts and work
splits the benchmark's configurations really run), against the CPU oracle.

The models keep the per-layer shape, vocabulary and GQA ratio of the configuration and fewer layers,
so that the oracle (weights held in fp32) fits the host and finishes in about a minute per case."""
import numpy as np
import pytest

from paper_2604_07609_b200 import binding as B
from synth import make_requests, make_weights, model_cfg, sched_cfg
from synth.workload import Request

from gpu_util import compare_with_oracle

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2     # max-abs logit error, bf16 mode


def _report(name, r):
    rows = max(sum(s[4] for s in rec["scheduled"]) for rec in r["trace"])
    dec = max(sum(1 for s in rec["scheduled"] if s[2] == 2) for rec in r["trace"])
    print(f"{name}: max-abs logit error {r['err']:.3e} (oracle with the data path's 16-bit rounding points), "
          f"{r['err_plain']:.3e} (plain high-precision oracle); {len(r['trace'])} iterations, up to {rows} rows "
          f"and {dec} decode rows per step, {r['n_margin']} token decisions inside the margin")
    assert r["err_plain"] <= TOL_BF16
    return rows, dec


def test_8b_layer_shape_small_sample_topk():
    """Four requests, prompts of at most 64 tokens, 16 new tokens each, top-k 50 at T 0.8: the sample
    the benchmark's CPU leg times, on four layers of the 8B shape (d 4096, 32/8 heads of 128, FFN
    14336, vocabulary 128256), streaming weight layout, tensor-core GEMMs."""
    model = model_cfg(3, n_layers=4)
    sched = sched_cfg(3, max_batch=256, prefill_chunk_tokens=512, n_blocks=256, n_slots=64, max_prompt=64, max_new=16)
    reqs = make_requests(3, n_requests=4)
    for r in reqs:
        r.prompt = r.prompt[:64]
        r.max_new = 16
    w = make_weights(model, 20260407, "cpu")
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, gemm_impl=B.GEMM_TC,
                            weights_layout=B.WEIGHTS_STREAMING)
    _report("8B layer shape, 4 requests", r)


def test_8b_layer_shape_128_row_decode_batch_and_multi_pass_prefill():
    """128 requests with contexts of 100 to 200 tokens on two layers of the 8B shape: prefill
    steps of more than 512 rows (three token passes, 256-column accumulators, generic stream-K ranges
    that cross weight tiles in gate/up and the LM head), then decode steps of 128 rows whose
    attention sub-ranges hold many tiles, whole and cut units alike."""
    model = model_cfg(3, n_layers=2)
    sched = sched_cfg(3, max_batch=128, prefill_chunk_tokens=512, n_blocks=2048, n_slots=256, max_prompt=256, max_new=4)
    rng = np.random.default_rng(31)
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 4)
            for t, p in enumerate(rng.integers(100, 201, size=128))]
    w = make_weights(model, 20260408, "cpu")
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, gemm_impl=B.GEMM_TC,
                            weights_layout=B.WEIGHTS_STREAMING)
    rows, dec = _report("8B layer shape, 128-row batch", r)
    assert rows > 512 and dec == 128


def test_1b_layer_shape_head_dim_64_four_heads_per_group():
    """Four layers of the 1B shape (d 2048, 32/8 heads of 64, FFN 8192, vocabulary 32000): the kernel
    instance with head_dim 64 and four query heads per kv head."""
    model = model_cfg(2, n_layers=4)
    sched = sched_cfg(2, max_batch=48, prefill_chunk_tokens=512, n_blocks=2048, n_slots=128, max_prompt=320, max_new=5)
    rng = np.random.default_rng(32)
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 5)
            for t, p in enumerate(rng.integers(40, 321, size=48))]
    w = make_weights(model, 20260409, "cpu")
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, gemm_impl=B.GEMM_TC,
                            weights_layout=B.WEIGHTS_STREAMING)
    rows, dec = _report("1B layer shape", r)
    assert dec == 48


def test_moe_layer_shape_two_layers():
    """Two layers of the routed-expert shape (8 experts of FFN 14336, top-2, d 4096, vocabulary 32000):
    the per-layer expert GEMM shapes of the full model."""
    model = model_cfg(5, n_layers=2)
    sched = sched_cfg(5, max_batch=16, prefill_chunk_tokens=64, n_blocks=256, n_slots=64, max_prompt=96, max_new=3)
    rng = np.random.default_rng(33)
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 3)
            for t, p in enumerate(rng.integers(8, 33, size=8))]
    w = make_weights(model, 20260410, "cpu")
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, gemm_impl=B.GEMM_TC,
                            weights_layout=B.WEIGHTS_STREAMING)
    _report("routed-expert layer shape", r)
