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
    rope_base: float = 0.0       # > 0: rotary position embedding on Q and K (half-split pairing) with this base

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


@dataclass(frozen=True)
class MlpConfig:
    """The feed-forward half of a transformer block on the same layout: pre-norm, up projection (with a gate
    projection for the gated variant), activation, down projection, optional residual."""
    name: str
    batch: int
    seq: int
    d_model: int
    d_ff: int
    dtype: str          # "fp32" or "bf16"
    norm: str           # "layernorm" or "rmsnorm"
    act: str            # "gelu" (tanh form, one up projection) or "swiglu" (silu(gate) * up)
    has_bias: bool
    residual: bool
    eps: float
    seed: int
    w_std: float

    @property
    def n_tokens(self) -> int:
        return self.batch * self.seq

    @property
    def gated(self) -> bool:
        return self.act == "swiglu"

    def flops(self) -> float:
        """Algorithmic forward+backward flops: each projection costs one product forward and two backward."""
        n_proj = 3 if self.gated else 2
        return 3.0 * n_proj * 2.0 * self.n_tokens * self.d_model * self.d_ff


MLP_CONFIGS = {
    # the paper's single-MatMul benchmark shapes (R-Tile ablation figure): forward (M=512, K=2048, N=8192) and the
    # backward product dA = dO B^T (M=512, K=8192, N=2048) are the up projection of this block and its input gradient
    "matmul-512x2048x8192": MlpConfig("mlp-matmul-512x2048x8192", 1, 512, 2048, 8192, "bf16", "layernorm", "gelu",
                                      True, True, 1e-5, 11, 0.02),
    # Llama-3.2-1B-shaped gated block (d_ff = 8192) behind the attention layer of workload 4
    "llama1b": MlpConfig("mlp-llama1b-swiglu", 2, 2048, 2048, 8192, "bf16", "rmsnorm", "swiglu", False, True, 1e-5, 12, 0.02),
    # GPT-2-small-shaped block (d_ff = 3072) behind the attention layer of workload 2
    "gpt2": MlpConfig("mlp-gpt2-small-gelu", 4, 512, 768, 3072, "bf16", "layernorm", "gelu", True, True, 1e-5, 13, 0.02),
}


@dataclass(frozen=True)
class XattnConfig:
    """A pre-norm cross-attention layer: queries from the normalised hidden states X [batch, seq, d_model], keys
    and values from a memory M [batch, seq_kv, d_mem] (an encoder's output, used as it is), no mask."""
    name: str
    batch: int
    seq: int            # query tokens per sequence
    seq_kv: int         # memory tokens per sequence
    d_model: int
    d_mem: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str
    norm: str
    has_bias: bool
    residual: bool
    eps: float
    seed: int
    w_std: float
    softmax_scale: float = 0.0
    causal: bool = False          # a memory position has no order relative to a query: never masked
    rope_base: float = 0.0

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

    def flops(self) -> float:
        """Algorithmic forward+backward flops: every projection once forward and twice backward, the two attention
        products once forward and four times backward (dV, dP, dQ, dK)."""
        nq, nk = self.batch * self.seq, self.batch * self.seq_kv
        proj = 2.0 * nq * self.d_model * self.d_q * 2 + 2.0 * nk * self.d_mem * self.d_kv * 2
        one_gemm = 2.0 * self.batch * self.n_q_heads * self.seq * self.seq_kv * self.head_dim
        return 3.0 * proj + 6.0 * one_gemm


XATTN_CONFIGS = {
    # Whisper-large-shaped decoder cross-attention (the paper's model table: Whisper-Large, batch 2): 20 heads of 64
    # over d_model 1280; 1500 encoder positions stand for 30 s of audio, 448 is the decoder's token limit
    "whisper-large": XattnConfig("xattn-whisper-large", 2, 448, 1500, 1280, 1280, 20, 20, 64, "bf16", "layernorm",
                                 True, True, 1e-5, 21, 0.02),
    # a small ragged case the oracle finishes in well under a second
    "tiny": XattnConfig("xattn-tiny-fp32", 2, 37, 75, 64, 96, 2, 1, 32, "fp32", "layernorm", True, True, 1e-5, 22, 0.05),
}
