"""Seeded random weights in the flat tensor order the library documents.

Tensor order inside the flat buffer (every tensor starts on a 256-byte
boundary; matrices are row-major [out_features, in_features]):

  id 0  embed    [V, d]                      model dtype
  id 1  wqkv     [L, (Hq+2*Hkv)*hd, d]       rows: q heads, k heads, v heads
  id 2  wo       [L, d, Hq*hd]
  id 3  wgu      [L, E', 2*F, d]             rows: gate [0,F), up [F,2F); E' = max(1, E)
  id 4  wd       [L, E', d, F]
  id 5  wr       [L, E, d]                   fp32 always (absent when E == 0)
  id 6  norm1    [L, d]                      fp32 always
  id 7  norm2    [L, d]                      fp32 always
  id 8  normf    [d]                         fp32 always
  id 9  lm_head  [V, d]                      model dtype

Values: N(0, 0.02) from a seeded torch generator, one stream per tensor id,
rounded once to the model dtype.  Norm gains are 1.0 unless `random_gains`.
No arithmetic of the serving method lives here.
"""
from __future__ import annotations

import numpy as np
import torch

from .configs import ModelCfg

TENSOR_NAMES = ["embed", "wqkv", "wo", "wgu", "wd", "wr", "norm1", "norm2", "normf", "lm_head"]
_ALIGN = 256


def _shapes(m: ModelCfg):
    E1 = max(1, m.n_experts)
    return {
        "embed": (m.vocab, m.d_model),
        "wqkv": (m.n_layers, m.qkv_dim, m.d_model),
        "wo": (m.n_layers, m.d_model, m.q_dim),
        "wgu": (m.n_layers, E1, 2 * m.d_ff, m.d_model),
        "wd": (m.n_layers, E1, m.d_model, m.d_ff),
        "wr": (m.n_layers, m.n_experts, m.d_model),
        "norm1": (m.n_layers, m.d_model),
        "norm2": (m.n_layers, m.d_model),
        "normf": (m.d_model,),
        "lm_head": (m.vocab, m.d_model),
    }


_FP32_ALWAYS = {"wr", "norm1", "norm2", "normf"}


def weight_layout(m: ModelCfg):
    """Return ({name: (byte_offset, shape, torch_dtype)}, total_bytes)."""
    wdt = torch.bfloat16 if m.dtype == "bf16" else torch.float32
    out = {}
    off = 0
    for name in TENSOR_NAMES:
        shape = _shapes(m)[name]
        dt = torch.float32 if name in _FP32_ALWAYS else wdt
        n = int(np.prod(shape))
        out[name] = (off, shape, dt)
        nbytes = n * (4 if dt == torch.float32 else 2)
        off += (nbytes + _ALIGN - 1) // _ALIGN * _ALIGN
    return out, off


def make_weights(m: ModelCfg, seed: int, device: str = "cpu", random_gains: bool = False,
                 std: float = 0.02) -> torch.Tensor:
    """Flat uint8 buffer on `device` holding all tensors in the documented order.

    The generator lives on `device`, so CPU- and CUDA-made buffers differ;
    whoever needs both views of the same weights makes them once and copies.
    """
    layout, total = weight_layout(m)
    buf = torch.zeros(total, dtype=torch.uint8, device=device)
    for tid, name in enumerate(TENSOR_NAMES):
        off, shape, dt = layout[name]
        n = int(np.prod(shape))
        if n == 0:
            continue
        esz = 4 if dt == torch.float32 else 2
        view = buf[off:off + n * esz].view(dt)
        g = torch.Generator(device=device)
        g.manual_seed((seed * 1000003 + tid) & 0x7FFFFFFFFFFF)
        if name in ("norm1", "norm2", "normf"):
            if random_gains:
                t = torch.empty(n, dtype=torch.float32, device=device)
                t.normal_(1.0, 0.1, generator=g)
                view.copy_(t)
            else:
                view.fill_(1.0)
            continue
        # draw in fp32 chunks to bound temporary memory on large models
        chunk = 1 << 26
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            t = torch.empty(e - s, dtype=torch.float32, device=device)
            t.normal_(0.0, std, generator=g)
            view[s:e].copy_(t)  # RNE to bf16 when the model dtype is bf16
    return buf


def weights_as_numpy(m: ModelCfg, buf: torch.Tensor, names=None, layers=None) -> dict:
    """Float32 numpy views (copies) of tensors in `buf`, exactly the stored values.

    `layers` optionally restricts per-layer tensors to the first `layers` layers
    (to keep host memory bounded on large shapes).
    """
    layout, _ = weight_layout(m)
    out = {}
    for name in (names or TENSOR_NAMES):
        off, shape, dt = layout[name]
        n = int(np.prod(shape))
        if n == 0:
            out[name] = np.zeros(shape, dtype=np.float32)
            continue
        esz = 4 if dt == torch.float32 else 2
        if layers is not None and len(shape) >= 2 and shape[0] == m.n_layers and name not in ("embed", "lm_head"):
            per = n // m.n_layers
            n = per * layers
            shape = (layers,) + tuple(shape[1:])
        t = buf[off:off + n * esz].view(dt).to(torch.float32).cpu().numpy().reshape(shape)
        out[name] = t
    return out
