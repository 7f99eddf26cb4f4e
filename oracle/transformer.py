"""Oracle O2: decoder-only transformer math (pre-norm, RMSNorm + RoPE + GQA + SwiGLU,
optional top-k-routed mixture of experts).  TEST INFRASTRUCTURE ONLY.

The paper treats the model as an opaque engine with paged KV cache, context
attention and a fused MLP / MoE plug-in (Sections 4.2, 4.3, 6.1); the math is the
standard one and is written here from its textbook definitions:

  n   = x / sqrt(mean(x^2) + eps) * g
  h  += Wo . Attn(RoPE(Wq n1), RoPE(Wk n1), Wv n1)      causal, scale 1/sqrt(hd),
                                                        q head j uses kv head j // (Hq/Hkv)
  h  += Wd . (silu(Wg n2) * (Wu n2))                    dense FFN
  h  += sum_e w_e . FFN_e(n2),  p = softmax(Wr n2), top-k experts (ties -> lower id),
        w_e = p_e / sum of the chosen p                  MoE FFN
  logits = Wlm . norm_f(h)

Two implementations live here and must agree: `forward_dense` (whole sequence at
once, contiguous K/V, no cache) and `PagedModel` (chunked steps over a block-paged
KV pool, driven by the scheduler oracle's block tables).

`act_round` models the reduced-precision storage points of the bf16 mode: values
are rounded to bf16 exactly where the bf16 data path stores 16-bit values (GEMM
operand inputs, the rotated queries handed to attention, and the KV pool; the
paper's engine runs its attention in 16-bit precision, Section 6.1); everything else stays in `dtype` (float64 by
default).  With act_round=None this is the pure high-precision reference.
"""
from __future__ import annotations

import numpy as np


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16, returned in the input's dtype."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    out = r.astype(np.uint32).view(np.float32)
    out = np.where(np.isnan(f), f, out)
    return out.astype(x.dtype, copy=False)


def rmsnorm(x, g, eps):
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope_angles(positions, head_dim, theta):
    """angle[p, i] = p * theta^(-2i/hd), i in [0, hd/2)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv = theta ** (-2.0 * i / head_dim)
    return np.asarray(positions, dtype=np.float64)[:, None] * inv[None, :]


def rope(x, positions, theta):
    """Rotate-half pairing: element i pairs with i + hd/2.  x: [T, H, hd]."""
    hd = x.shape[-1]
    ang = rope_angles(positions, hd, theta)
    c = np.cos(ang).astype(np.float32).astype(x.dtype)[:, None, :]   # tables are kept in fp32
    s = np.sin(ang).astype(np.float32).astype(x.dtype)[:, None, :]
    x1, x2 = x[..., : hd // 2], x[..., hd // 2:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def softmax(x, axis=-1):
    m = np.max(x, axis=axis, keepdims=True)
    e = np.exp(x - m)
    return e / np.sum(e, axis=axis, keepdims=True)


def attention_rows(q, k, v, q_pos, n_rep):
    """q: [Tq, Hq, hd] at absolute positions q_pos; k, v: [Tk, Hkv, hd] at positions
    0..Tk-1.  Row t attends to keys at positions <= q_pos[t].  Returns [Tq, Hq, hd]."""
    Tq, Hq, hd = q.shape
    Tk = k.shape[0]
    out = np.zeros_like(q)
    scale = 1.0 / np.sqrt(hd)
    kpos = np.arange(Tk)
    for h in range(Hq):
        g = h // n_rep
        s = (q[:, h, :] @ k[:, g, :].T) * scale                # [Tq, Tk]
        mask = kpos[None, :] > np.asarray(q_pos)[:, None]
        s = np.where(mask, -np.inf, s)
        p = softmax(s, axis=-1)
        out[:, h, :] = p @ v[:, g, :]
    return out


class Weights:
    """Named float arrays (already holding the stored, possibly bf16-rounded values)."""

    def __init__(self, cfg, arrays: dict, dtype=np.float64):
        self.cfg = cfg
        self.dtype = dtype
        self.a = {k: np.asarray(v, dtype=dtype) for k, v in arrays.items()}

    def __getitem__(self, k):
        return self.a[k]


def _ffn_dense(n2, wgu, wd, F, rb):
    gu = n2 @ wgu.T
    act = silu(gu[:, :F]) * gu[:, F:]
    return rb(act) @ wd.T


def _ffn(cfg, W, layer, n2_raw, rb):
    """n2_raw: normed input in working precision.  Returns the FFN output [T, d]."""
    F = cfg.d_ff
    n2 = rb(n2_raw)
    if cfg.n_experts == 0:
        return _ffn_dense(n2, W["wgu"][layer, 0], W["wd"][layer, 0], F, rb), None
    # router runs on the unrounded normed activations with fp32-stored router weights
    p = softmax(n2_raw @ W["wr"][layer].T, axis=-1)               # [T, E]
    T = n2.shape[0]
    k = cfg.top_k_experts
    out = np.zeros((T, cfg.d_model), dtype=n2.dtype)
    chosen = np.zeros((T, k), dtype=np.int64)
    for t in range(T):
        # top-k by (p desc, expert id asc)
        order = sorted(range(cfg.n_experts), key=lambda e: (-p[t, e], e))[:k]
        chosen[t] = order
        z = sum(p[t, e] for e in order)
        # fixed combine order: ascending expert id
        for e in sorted(order):
            y = _ffn_dense(n2[t:t + 1], W["wgu"][layer, e], W["wd"][layer, e], F, rb)
            out[t] += (p[t, e] / z) * y[0]
    return out, chosen


def forward_dense(cfg, W: Weights, tokens, act_round=None, return_hidden=False):
    """Whole sequence at once, contiguous K/V, no cache.  Returns logits [T, V]."""
    rb = (lambda x: x) if act_round is None else act_round
    T = len(tokens)
    pos = np.arange(T)
    h = W["embed"][np.asarray(tokens)].astype(W.dtype)
    n_rep = cfg.n_q_heads // cfg.n_kv_heads
    for l in range(cfg.n_layers):
        n1 = rb(rmsnorm(h, W["norm1"][l], cfg.rms_eps))
        qkv = n1 @ W["wqkv"][l].T
        q = qkv[:, : cfg.q_dim].reshape(T, cfg.n_q_heads, cfg.head_dim)
        k = qkv[:, cfg.q_dim: cfg.q_dim + cfg.kv_dim].reshape(T, cfg.n_kv_heads, cfg.head_dim)
        v = qkv[:, cfg.q_dim + cfg.kv_dim:].reshape(T, cfg.n_kv_heads, cfg.head_dim)
        q = rb(rope(q, pos, cfg.rope_theta))       # q is a 16-bit operand of the attention contraction
        k = rb(rope(k, pos, cfg.rope_theta))       # K/V are stored in the cache dtype
        v = rb(v)
        a = attention_rows(q, k, v, pos, n_rep).reshape(T, cfg.q_dim)
        h = h + rb(a) @ W["wo"][l].T
        f, _ = _ffn(cfg, W, l, rmsnorm(h, W["norm2"][l], cfg.rms_eps), rb)
        h = h + f
    nf = rb(rmsnorm(h, W["normf"], cfg.rms_eps))
    logits = nf @ W["lm_head"].T
    return (logits, h) if return_hidden else logits


class PagedModel:
    """Chunked prefill + decode over a block-paged KV pool.

    Pool layout follows the KV layout of the data path in spirit only (indexing by
    physical block, kv head, in-block offset); `step` consumes the scheduler
    oracle's ScheduledItem list."""

    def __init__(self, cfg, W: Weights, n_blocks: int, block: int = 16, act_round=None):
        self.cfg, self.W, self.block = cfg, W, block
        self.rb = (lambda x: x) if act_round is None else act_round
        shp = (cfg.n_layers, n_blocks, block, cfg.n_kv_heads, cfg.head_dim)
        self.kpool = np.full(shp, np.nan, dtype=W.dtype)   # NaN poison: reading an unwritten cell shows
        self.vpool = np.full(shp, np.nan, dtype=W.dtype)
        self.last_routing = None

    def _gather(self, pool, l, table, n):
        blk = self.block
        rows = [pool[l, table[p // blk], p % blk] for p in range(n)]
        return np.stack(rows, axis=0)          # [n, Hkv, hd]

    def step(self, items):
        """items: scheduler ScheduledItem list with input_tokens.  Returns logits
        [n_sample_rows, V] in item order."""
        cfg, W, rb = self.cfg, self.W, self.rb
        toks, pos, owner = [], [], []
        for it in items:
            assert it.input_tokens is not None and len(it.input_tokens) == it.n_tokens
            toks += list(it.input_tokens)
            pos += list(range(it.start_pos, it.start_pos + it.n_tokens))
            owner += [it] * it.n_tokens
        T = len(toks)
        pos = np.asarray(pos)
        h = W["embed"][np.asarray(toks)].astype(W.dtype)
        n_rep = cfg.n_q_heads // cfg.n_kv_heads
        routing = []
        for l in range(cfg.n_layers):
            n1 = rb(rmsnorm(h, W["norm1"][l], cfg.rms_eps))
            qkv = n1 @ W["wqkv"][l].T
            q = qkv[:, : cfg.q_dim].reshape(T, cfg.n_q_heads, cfg.head_dim)
            k = qkv[:, cfg.q_dim: cfg.q_dim + cfg.kv_dim].reshape(T, cfg.n_kv_heads, cfg.head_dim)
            v = qkv[:, cfg.q_dim + cfg.kv_dim:].reshape(T, cfg.n_kv_heads, cfg.head_dim)
            q = rb(rope(q, pos, cfg.rope_theta))
            k = rb(rope(k, pos, cfg.rope_theta))
            v = rb(v)
            # write this step's K/V into the pool at block_table[pos // block], pos % block
            for t in range(T):
                it = owner[t]
                b = it.block_table[pos[t] // self.block]
                self.kpool[l, b, pos[t] % self.block] = k[t]
                self.vpool[l, b, pos[t] % self.block] = v[t]
            a = np.zeros((T, cfg.n_q_heads, cfg.head_dim), dtype=W.dtype)
            r0 = 0
            for it in items:
                n_ctx = it.start_pos + it.n_tokens
                kk = self._gather(self.kpool, l, it.block_table, n_ctx)
                vv = self._gather(self.vpool, l, it.block_table, n_ctx)
                rows = slice(r0, r0 + it.n_tokens)
                a[rows] = attention_rows(q[rows], kk, vv, pos[rows], n_rep)
                r0 += it.n_tokens
            h = h + rb(a.reshape(T, cfg.q_dim)) @ W["wo"][l].T
            f, ch = _ffn(cfg, W, l, rmsnorm(h, W["norm2"][l], cfg.rms_eps), rb)
            routing.append(ch)
            h = h + f
        self.last_routing = routing
        # LM head on sample rows only
        rows, r0 = [], 0
        for it in items:
            if it.sample:
                rows.append(r0 + it.n_tokens - 1)
            r0 += it.n_tokens
        if not rows:
            return np.zeros((0, cfg.vocab), dtype=W.dtype)
        nf = rb(rmsnorm(h[rows], W["normf"], cfg.rms_eps))
        return nf @ W["lm_head"].T
