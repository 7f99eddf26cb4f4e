"""GPU parity at the layer shapes that are benchmarked (the kernel instances, tile counts and work
splits the benchmark's configurations really run), against the CPU oracle.

The models keep the per-layer shape, vocabulary and GQA ratio of the configuration and fewer layers,
so that the oracle (weights held in fp32) fits the host and finishes in about a minute per case.

Tolerance at these shapes.  With d_model 4096 and N(0, 0.02) weights the logits have a standard
deviation of 1.28 and the 16-bit roundings of the data path alone move them by 5e-2 (one layer) to
1e-1 (four layers) in max-abs over the 128256 entries of a row: that is the distance between the two
CPU oracles, which differ only in the rounding hook.  The 2e-2 bound of the small configuration is
below that noise, so these tests state the bound relative to it (see compare_with_oracle): the GPU
must be at least as close to the rounding oracle as the plain oracle is, and about as close to the
plain oracle as the rounding oracle is.  A wrong tile, a dropped partial sum or a stale operand moves
logits by their full size (about 1) and fails by a factor of ten or more."""
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
    print(f"{name}: logits std {r['logit_std']:.2f}; gpu vs rounding oracle max {r['err']:.3e} rms {r['err_rms']:.3e}; "
          f"gpu vs plain oracle max {r['err_plain']:.3e} rms {r['err_plain_rms']:.3e}; rounding vs plain oracle max "
          f"{r['noise_max']:.3e} rms {r['noise_rms']:.3e}; {len(r['trace'])} iterations, up to {rows} rows and {dec} decode "
          f"rows per step, {r['n_margin']} token decisions inside the margin")
    return rows, dec


@pytest.mark.parametrize("gemm,fusion", [(B.GEMM_TC_PAIR, B.FUSION_OFF), (B.GEMM_TC, B.FUSION_OFF), (B.GEMM_TC, B.FUSION_ON)],
                         ids=["cta-pairs", "single-cta", "single-cta-fused-epilogues"])
def test_8b_layer_shape_small_sample_topk(gemm, fusion):
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
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, noise_relative=True, gemm_impl=gemm,
                            weights_layout=B.WEIGHTS_STREAMING, epilogue_fusion=fusion)
    _report("8B layer shape, 4 requests", r)


def test_8b_layer_shape_128_row_decode_batch_and_multi_pass_prefill():
    """128 requests with contexts of 100 to 200 tokens on two layers of the 8B shape.  The prefill
    budget is large here (4096 tokens), so the prompts are through in five steps of several thousand
    rows (many token passes per weight tile) and all 128 requests then decode together: steps of
    exactly 128 rows (128-column accumulators shared by the two epilogue groups, generic stream-K
    ranges that cross weight tiles in gate/up and the LM head) whose attention sub-ranges hold many
    tiles, whole and cut units alike."""
    model = model_cfg(3, n_layers=2)
    sched = sched_cfg(3, max_batch=128, prefill_chunk_tokens=4096, n_blocks=2048, n_slots=256, max_prompt=256, max_new=7)
    rng = np.random.default_rng(31)
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 7)
            for t, p in enumerate(rng.integers(100, 201, size=128))]
    w = make_weights(model, 20260408, "cpu")
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, noise_relative=True, gemm_impl=B.GEMM_AUTO,
                            weights_layout=B.WEIGHTS_STREAMING)
    rows, dec = _report("8B layer shape, 128-row batch", r)
    assert rows > 4096 and dec == 128


def test_1b_layer_shape_head_dim_64_four_heads_per_group():
    """Four layers of the 1B shape (d 2048, 32/8 heads of 64, FFN 8192, vocabulary 32000): the kernel
    instance with head_dim 64 and four query heads per kv head."""
    model = model_cfg(2, n_layers=4)
    sched = sched_cfg(2, max_batch=48, prefill_chunk_tokens=2048, n_blocks=2048, n_slots=128, max_prompt=320, max_new=8)
    rng = np.random.default_rng(32)
    reqs = [Request(t, 0.0, rng.integers(0, model.vocab, size=int(p)).astype(np.int32), 8)
            for t, p in enumerate(rng.integers(40, 321, size=48))]
    w = make_weights(model, 20260409, "cpu")
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, noise_relative=True, gemm_impl=B.GEMM_AUTO,
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
    r = compare_with_oracle(model, sched, reqs, w, TOL_BF16, oracle_dtype=np.float32, noise_relative=True, gemm_impl=B.GEMM_AUTO,
                            weights_layout=B.WEIGHTS_STREAMING)
    _report("routed-expert layer shape", r)
