"""Pins for the transformer oracle: library cross-checks on tiny shapes (torch CPU
ops as the textbook reference), special cases, and paged == dense."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import scheduler as O1
from oracle import transformer as O2
from synth import ModelCfg, make_weights, weights_as_numpy

TINY = ModelCfg(2, 64, 4, 2, 16, 96, 50, dtype="fp32")
TINY_MOE = ModelCfg(2, 64, 4, 2, 16, 48, 50, n_experts=4, top_k_experts=2, dtype="fp32")


def _weights(cfg, seed=1, random_gains=True, std=0.08):
    buf = make_weights(cfg, seed, "cpu", random_gains=random_gains, std=std)
    return O2.Weights(cfg, weights_as_numpy(cfg, buf))


def test_round_bf16_matches_torch():
    x = np.random.default_rng(0).normal(size=5000).astype(np.float32) * 3
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]      # exact ties: round to even
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O2.round_bf16(x), ref)
    assert O2.round_bf16(x.astype(np.float64)).dtype == np.float64


def test_rmsnorm_matches_torch():
    x = np.random.default_rng(1).normal(size=(5, 64))
    g = np.random.default_rng(2).normal(size=64)
    ref = F.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(g), 1e-5).numpy()
    assert np.allclose(O2.rmsnorm(x, g, 1e-5), ref, atol=1e-12)


def test_silu_softmax_match_torch():
    x = np.random.default_rng(3).normal(size=(4, 9)) * 4
    assert np.allclose(O2.silu(x), F.silu(torch.from_numpy(x)).numpy(), atol=1e-12)
    assert np.allclose(O2.softmax(x), torch.softmax(torch.from_numpy(x), -1).numpy(), atol=1e-12)
    assert np.allclose(O2.softmax(x).sum(-1), 1.0)


def test_rope_properties():
    x = np.random.default_rng(4).normal(size=(6, 3, 16))
    assert np.allclose(O2.rope(x, np.zeros(6), 10000.0), x)                      # identity at position 0
    y = O2.rope(x, np.arange(6) + 3, 10000.0)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-6)   # rotation
    # relative-position property: <rope(q,m), rope(k,n)> depends on m - n only
    q, k = x[:1], x[1:2]
    a = np.sum(O2.rope(q, [5], 1e4) * O2.rope(k, [2], 1e4))
    b = np.sum(O2.rope(q, [9], 1e4) * O2.rope(k, [6], 1e4))
    assert abs(a - b) < 1e-5
    # explicit complex-rotation definition for one pair (i, i + hd/2)
    p, i, hd = 7, 3, 16
    ang = p * 10000.0 ** (-2 * i / hd)
    z = (x[0, 0, i] + 1j * x[0, 0, i + hd // 2]) * np.exp(1j * ang)
    yy = O2.rope(x[:1], [p], 1e4)[0, 0]
    assert abs(yy[i] - z.real) < 1e-6 and abs(yy[i + hd // 2] - z.imag) < 1e-6


def test_attention_matches_torch_sdpa_causal_gqa():
    rng = np.random.default_rng(5)
    T, Hq, Hkv, hd = 9, 4, 2, 16
    q, k, v = rng.normal(size=(T, Hq, hd)), rng.normal(size=(T, Hkv, hd)), rng.normal(size=(T, Hkv, hd))
    out = O2.attention_rows(q, k, v, np.arange(T), Hq // Hkv)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    tv = torch.from_numpy(v).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.allclose(out, ref, atol=1e-10)
    # a single key reduces attention to V
    o1 = O2.attention_rows(q[:1], k[:1], v[:1], [0], 2)
    assert np.allclose(o1[0, 3], v[0, 1])


def _torch_forward(cfg, W, tokens):
    """Independent restatement with torch library ops (fp64)."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    T = len(tokens)
    h = t(W["embed"])[torch.tensor(tokens)]
    hd = cfg.head_dim
    inv = cfg.rope_theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
    ang = torch.arange(T, dtype=torch.float64)[:, None] * inv[None]
    cos, sin = torch.cos(ang).float().double(), torch.sin(ang).float().double()

    def rot(x):  # [T, H, hd]
        x1, x2 = x[..., : hd // 2], x[..., hd // 2:]
        return torch.cat([x1 * cos[:, None] - x2 * sin[:, None], x2 * cos[:, None] + x1 * sin[:, None]], -1)

    for l in range(cfg.n_layers):
        n1 = F.rms_norm(h, (cfg.d_model,), t(W["norm1"][l]), cfg.rms_eps)
        qkv = F.linear(n1, t(W["wqkv"][l]))
        q = rot(qkv[:, :cfg.q_dim].view(T, cfg.n_q_heads, hd))
        k = rot(qkv[:, cfg.q_dim:cfg.q_dim + cfg.kv_dim].view(T, cfg.n_kv_heads, hd))
        v = qkv[:, cfg.q_dim + cfg.kv_dim:].view(T, cfg.n_kv_heads, hd)
        rep = cfg.n_q_heads // cfg.n_kv_heads
        a = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None],
                                           k.permute(1, 0, 2)[None].repeat_interleave(rep, 1),
                                           v.permute(1, 0, 2)[None].repeat_interleave(rep, 1),
                                           is_causal=True)[0].permute(1, 0, 2).reshape(T, cfg.q_dim)
        h = h + F.linear(a, t(W["wo"][l]))
        n2 = F.rms_norm(h, (cfg.d_model,), t(W["norm2"][l]), cfg.rms_eps)
        if cfg.n_experts == 0:
            gu = F.linear(n2, t(W["wgu"][l, 0]))
            h = h + F.linear(F.silu(gu[:, :cfg.d_ff]) * gu[:, cfg.d_ff:], t(W["wd"][l, 0]))
        else:
            p = torch.softmax(F.linear(n2, t(W["wr"][l])), -1)
            top, idx = torch.topk(p, cfg.top_k_experts, dim=-1)
            wts = top / top.sum(-1, keepdim=True)
            y = torch.zeros_like(h)
            for e in range(cfg.n_experts):
                gu = F.linear(n2, t(W["wgu"][l, e]))
                fe = F.linear(F.silu(gu[:, :cfg.d_ff]) * gu[:, cfg.d_ff:], t(W["wd"][l, e]))
                sel = (idx == e).to(torch.float64) * wts
                y = y + sel.sum(-1, keepdim=True) * fe
            h = h + y
    nf = F.rms_norm(h, (cfg.d_model,), t(W["normf"]), cfg.rms_eps)
    return F.linear(nf, t(W["lm_head"])).numpy()


@pytest.mark.parametrize("cfg", [TINY, TINY_MOE], ids=["dense", "moe"])
def test_forward_dense_matches_torch_restatement(cfg):
    W = _weights(cfg)
    tokens = list(np.random.default_rng(6).integers(0, cfg.vocab, size=11))
    ours = O2.forward_dense(cfg, W, tokens)
    ref = _torch_forward(cfg, W, tokens)
    assert np.abs(ours - ref).max() < 1e-9


def test_gqa_with_equal_heads_is_mha_and_zero_weights():
    cfg = TINY.with_(n_kv_heads=4)
    W = _weights(cfg)
    tokens = [1, 2, 3, 4, 5]
    a = O2.forward_dense(cfg, W, tokens)
    assert np.abs(a - _torch_forward(cfg, W, tokens)).max() < 1e-9
    # with Wo = Wd = 0 every block is the identity: logits = Wlm . norm_f(embed)
    W.a["wo"] = np.zeros_like(W["wo"]); W.a["wd"] = np.zeros_like(W["wd"])
    z = O2.forward_dense(cfg, W, tokens)
    ref = O2.rmsnorm(W["embed"][tokens], W["normf"], cfg.rms_eps) @ W["lm_head"].T
    assert np.allclose(z, ref, atol=1e-12)


def test_moe_special_cases():
    # identical experts == dense FFN whatever the routing; weights sum to one
    cfg = TINY_MOE
    W = _weights(cfg)
    for e in range(1, cfg.n_experts):
        W.a["wgu"][:, e] = W["wgu"][:, 0]
        W.a["wd"][:, e] = W["wd"][:, 0]
    dense = cfg.with_(n_experts=0, top_k_experts=0)
    Wd = O2.Weights(dense, {k: (v[:, :1] if k in ("wgu", "wd") else v) for k, v in W.a.items()})
    tokens = [3, 1, 4, 1, 5, 9, 2, 6]
    assert np.abs(O2.forward_dense(cfg, W, tokens) - O2.forward_dense(dense, Wd, tokens)).max() < 1e-10
    # one expert, top-1 == dense
    one = cfg.with_(n_experts=1, top_k_experts=1)
    W1 = O2.Weights(one, {k: (v[:, :1] if k in ("wgu", "wd", "wr") else v) for k, v in W.a.items()})
    assert np.abs(O2.forward_dense(one, W1, tokens) - O2.forward_dense(dense, Wd, tokens)).max() < 1e-10


def _paged_logits(cfg, W, prompt, chunk, n_blocks=12, perm=None, block=4, act_round=None):
    """Prefill `prompt` in chunks through the paged model using the scheduler oracle's tables."""
    sch = O1.Scheduler([O1.SimRequest(0, len(prompt), 1, -1, prompt)], 2, chunk, n_blocks, block)
    if perm is not None:
        sch.stack = [perm[b] for b in sch.stack]
    model = O2.PagedModel(cfg, W, n_blocks, block, act_round)
    rows = []
    while True:
        items = sch.begin(0)
        if items is None:
            break
        lg = model.step(items)
        sch.finish(items, [0] * len(lg))
        if len(lg):
            rows.append(lg[0])
    return rows[-1]


@pytest.mark.parametrize("cfg", [TINY, TINY_MOE], ids=["dense", "moe"])
def test_paged_chunked_equals_dense_unpaged(cfg):
    W = _weights(cfg)
    prompt = [int(x) for x in np.random.default_rng(7).integers(0, cfg.vocab, size=19)]
    dense_last = O2.forward_dense(cfg, W, prompt)[-1]
    perm = list(np.random.default_rng(8).permutation(12))
    for chunk in (1, 7, 19, 64):
        for pm in (None, perm):
            got = _paged_logits(cfg, W, prompt, chunk, perm=pm)
            assert np.abs(got - dense_last).max() < 1e-5


def test_paged_decode_equals_dense_on_extended_sequence():
    cfg = TINY
    W = _weights(cfg)
    rng = np.random.default_rng(9)
    prompt = [int(x) for x in rng.integers(0, cfg.vocab, size=10)]
    forced = [int(x) for x in rng.integers(0, cfg.vocab, size=6)]
    sch = O1.Scheduler([O1.SimRequest(0, 10, 6, -1, prompt)], 2, 4, 16, 4)
    model = O2.PagedModel(cfg, W, 16, 4)
    got, k = [], 0
    while True:
        items = sch.begin(0)
        if items is None:
            break
        lg = model.step(items)
        if len(lg):
            got.append(lg[0]); sch.finish(items, [forced[k]]); k += 1
        else:
            sch.finish(items, [])
    full = O2.forward_dense(cfg, W, prompt + forced[:-1])
    for j in range(6):
        assert np.abs(got[j] - full[9 + j]).max() < 1e-9


def test_bf16_rounding_mode_paged_equals_dense_and_differs_from_exact():
    cfg = TINY
    W = _weights(cfg)
    prompt = [int(x) for x in np.random.default_rng(10).integers(0, cfg.vocab, size=13)]
    d = O2.forward_dense(cfg, W, prompt, act_round=O2.round_bf16)[-1]
    p = _paged_logits(cfg, W, prompt, 5, act_round=O2.round_bf16)
    assert np.abs(d - p).max() < 1e-9     # same rounding points => identical up to summation order
    exact = O2.forward_dense(cfg, W, prompt)[-1]
    assert 1e-6 < np.abs(d - exact).max() < 5e-2
