"""Model and scheduler shapes of the five benchmark configurations.

Shapes only; no arithmetic of the method lives here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ModelCfg:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    n_experts: int = 0          # 0 = dense FFN
    top_k_experts: int = 0
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5
    dtype: str = "bf16"         # "bf16" | "fp32" (reference mode)

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def qkv_dim(self) -> int:
        return self.q_dim + 2 * self.kv_dim

    def with_(self, **kw) -> "ModelCfg":
        return replace(self, **kw)


@dataclass(frozen=True)
class SchedCfg:
    max_batch: int
    prefill_chunk_tokens: int
    block_size: int = 16
    n_blocks: int = 256
    n_slots: int = 4096
    max_prompt: int = 4096
    max_new: int = 1024

    def with_(self, **kw) -> "SchedCfg":
        return replace(self, **kw)


# index -> (model, sched, stream description)
CONFIGS = {
    1: dict(
        name="C1-tiny",
        model=ModelCfg(2, 256, 4, 4, 64, 1024, 4096, rope_theta=10000.0),
        sched=SchedCfg(max_batch=8, prefill_chunk_tokens=64, n_blocks=256, n_slots=64,
                       max_prompt=64, max_new=32),
    ),
    2: dict(
        name="C2-1B",
        model=ModelCfg(16, 2048, 32, 8, 64, 8192, 32000, rope_theta=10000.0),
        sched=SchedCfg(max_batch=128, prefill_chunk_tokens=512, n_blocks=16384, n_slots=4096,
                       max_prompt=1024, max_new=512),
    ),
    3: dict(
        name="C3-8B",
        model=ModelCfg(32, 4096, 32, 8, 128, 14336, 128256, rope_theta=500000.0),
        sched=SchedCfg(max_batch=256, prefill_chunk_tokens=512, n_blocks=0, n_slots=4096,
                       max_prompt=4096, max_new=1024),
    ),
    4: dict(
        name="C4-8B-interference",
        model=ModelCfg(32, 4096, 32, 8, 128, 14336, 128256, rope_theta=500000.0),
        sched=SchedCfg(max_batch=256, prefill_chunk_tokens=512, n_blocks=0, n_slots=4096,
                       max_prompt=4096, max_new=1024),
    ),
    5: dict(
        name="C5-MoE",
        model=ModelCfg(32, 4096, 32, 8, 128, 14336, 32000, n_experts=8, top_k_experts=2,
                       rope_theta=1e6),
        sched=SchedCfg(max_batch=256, prefill_chunk_tokens=512, n_blocks=0, n_slots=4096,
                       max_prompt=2048, max_new=512),
    ),
}


def model_cfg(idx: int, **kw) -> ModelCfg:
    m = CONFIGS[idx]["model"]
    return m.with_(**kw) if kw else m


def sched_cfg(idx: int, **kw) -> SchedCfg:
    s = CONFIGS[idx]["sched"]
    return s.with_(**kw) if kw else s
