"""The five synthetic attention-layer workloads and helpers to derive reduced ones.

Each stands in for one of the transformer workloads the paper evaluates (its model
table lists decoder-only LLMs at 512 tokens, BERT/ViT encoders, and attention
shapes [seq, heads, hidden] such as (512, 32, 2048)); no dataset or checkpoint is
involved, every tensor is drawn from a seeded normal distribution.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class LayerConfig:
    name: str
    batch: int
    seq: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str          # "fp32" or "bf16" (bf16 storage, fp32 accumulation)
    norm: str           # "layernorm" or "rmsnorm"
    causal: bool
    has_bias: bool
    residual: bool
    eps: float
    seed: int
    w_std: float
    softmax_scale: float = 0.0   # <= 0 means 1/sqrt(head_dim)

    @property
    def n_tokens(self) -> int:
        return self.batch * self.seq

    @property
    def d_q(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def scale(self) -> float:
        return self.softmax_scale if self.softmax_scale > 0 else self.head_dim ** -0.5

    def flops(self, recompute: bool = False) -> float:
        """Algorithmic forward+backward flops (multiply-add = 2).

        Causal attention counts only the T(T+1)/2 unmasked pairs.  With
        ``recompute`` the backward's second evaluation of the scores is added.
        """
        n = self.n_tokens
        proj = 2.0 * n * self.d_model * (self.d_q + 2 * self.d_kv) + 2.0 * n * self.d_q * self.d_model
        pairs = self.seq * (self.seq + 1) / 2 if self.causal else float(self.seq) * self.seq
        one_gemm = 2.0 * self.batch * self.n_q_heads * pairs * self.head_dim
        total = 3.0 * proj + 6.0 * one_gemm
        if recompute:
            total += one_gemm
        return total


CONFIGS = {
    1: LayerConfig("cfg1-tiny-fp32", 1, 64, 64, 2, 2, 32, "fp32", "layernorm", True, False, False, 1e-5, 0, 0.02),
    2: LayerConfig("cfg2-gpt2-small", 4, 512, 768, 12, 12, 64, "bf16", "layernorm", True, True, False, 1e-5, 1, 0.02),
    3: LayerConfig("cfg3-vit-base", 32, 197, 768, 12, 12, 64, "bf16", "layernorm", False, False, False, 1e-6, 2, 0.02),
    4: LayerConfig("cfg4-llama1b-gqa", 2, 2048, 2048, 32, 8, 64, "bf16", "rmsnorm", True, False, False, 1e-5, 3, 0.02),
    5: LayerConfig("cfg5-llama7b-long", 1, 8192, 4096, 32, 32, 128, "bf16", "rmsnorm", True, False, False, 1e-5, 4, 0.01),
}


def get_config(i: int) -> LayerConfig:
    return CONFIGS[i]


def scaled_config(cfg: LayerConfig, **kw) -> LayerConfig:
    """A copy of ``cfg`` with some fields replaced (smaller batch, other flags...)."""
    return replace(cfg, **kw)
