"""Counter-based normal generator: value = g(seed, tensor id, element index).

Each element is a pure function of its key, so any slice of any tensor can be
regenerated on its own and both sides of a parity test see identical inputs.
Values are rounded to the storage dtype (fp32 or bf16, round-to-nearest-even)
before anyone uses them; the oracle receives those rounded values as float64.
"""
from __future__ import annotations

import numpy as np

from .configs import LayerConfig

TENSOR_IDS = {
    "X": 0, "Wq": 1, "Wk": 2, "Wv": 3, "Wo": 4,
    "bq": 5, "bk": 6, "bv": 7, "bo": 8, "gamma": 9, "beta": 10, "dY": 11,
    "W1": 12, "Wg": 13, "W2": 14, "b1": 15, "bg": 16, "b2": 17,
    "Aq": 18, "Ak": 19, "Av": 20, "Bq": 21, "Bk": 22, "Bv": 23,
    "M": 24,
}

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    z = (z + np.uint64(0x9E3779B97F4A7C15))
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def normal_f64(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """``count`` standard normals for element indices ``start .. start+count-1``."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64)
        key = _splitmix64(np.uint64(seed) * np.uint64(0xD1342543DE82EF95)
                          + np.uint64(tensor_id) * np.uint64(0xA0761D6478BD642F) + np.uint64(1))
        a = _splitmix64(key ^ (idx * np.uint64(2)))
        b = _splitmix64(key ^ (idx * np.uint64(2) + np.uint64(1)))
    # 53-bit uniforms; u1 in (0, 1], u2 in [0, 1)
    u1 = ((a >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
    u2 = (b >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float64 values to the storage dtype and return them as float64."""
    x32 = x.astype(np.float32)
    if dtype == "fp32":
        return x32.astype(np.float64)
    if dtype == "bf16":
        bits = to_bf16_bits(x32).astype(np.uint32) << np.uint32(16)
        return bits.view(np.float32).reshape(x.shape).astype(np.float64)
    raise ValueError(dtype)


def make_inputs(cfg: LayerConfig, *, affine_noise: bool = False) -> dict:
    """All layer inputs for ``cfg`` as float64 arrays holding storage-rounded values.

    Matrices are rounded to ``cfg.dtype``; vectors (gamma, beta, biases) are fp32 in
    both dtypes.  ``affine_noise`` draws gamma ~ 1 + 0.1 N(0,1) and beta ~ 0.1 N(0,1)
    instead of the identity affine the workloads specify, so that those code paths
    are exercised away from 1 and 0.
    """
    s = cfg.seed
    n, d, dq, dkv = cfg.n_tokens, cfg.d_model, cfg.d_q, cfg.d_kv

    def mat(name, shape, std):
        cnt = int(np.prod(shape))
        v = normal_f64(s, TENSOR_IDS[name], 0, cnt).reshape(shape) * std
        return round_to_storage(v, cfg.dtype)

    def vec(name, length, std, mean=0.0):
        v = normal_f64(s, TENSOR_IDS[name], 0, length) * std + mean
        return v.astype(np.float32).astype(np.float64)

    out = {
        "X": mat("X", (cfg.batch, cfg.seq, d), 1.0),
        "dY": mat("dY", (cfg.batch, cfg.seq, d), 1.0),
        "Wq": mat("Wq", (d, dq), cfg.w_std),
        "Wk": mat("Wk", (d, dkv), cfg.w_std),
        "Wv": mat("Wv", (d, dkv), cfg.w_std),
        "Wo": mat("Wo", (dq, d), cfg.w_std),
    }
    if affine_noise:
        out["gamma"] = vec("gamma", d, 0.1, 1.0)
        out["beta"] = vec("beta", d, 0.1) if cfg.norm == "layernorm" else None
    else:
        out["gamma"] = np.ones(d)
        out["beta"] = np.zeros(d) if cfg.norm == "layernorm" else None
    if cfg.has_bias:
        out["bq"] = vec("bq", dq, cfg.w_std)
        out["bk"] = vec("bk", dkv, cfg.w_std)
        out["bv"] = vec("bv", dkv, cfg.w_std)
        out["bo"] = vec("bo", d, cfg.w_std)
    else:
        out["bq"] = out["bk"] = out["bv"] = out["bo"] = None
    return out


def make_mlp_inputs(cfg, *, affine_noise: bool = False) -> dict:
    """All inputs of the feed-forward block ``cfg`` (an ``MlpConfig``) as float64 arrays of storage-rounded values:
    X, dY ~ N(0, 1); W1, Wg [d_model, d_ff] and W2 [d_ff, d_model] ~ N(0, w_std^2); vectors are fp32."""
    s = cfg.seed
    d, f = cfg.d_model, cfg.d_ff

    def mat(name, shape, std):
        cnt = int(np.prod(shape))
        return round_to_storage(normal_f64(s, TENSOR_IDS[name], 0, cnt).reshape(shape) * std, cfg.dtype)

    def vec(name, length, std, mean=0.0):
        return (normal_f64(s, TENSOR_IDS[name], 0, length) * std + mean).astype(np.float32).astype(np.float64)

    out = {"X": mat("X", (cfg.batch, cfg.seq, d), 1.0), "dY": mat("dY", (cfg.batch, cfg.seq, d), 1.0),
           "W1": mat("W1", (d, f), cfg.w_std), "W2": mat("W2", (f, d), cfg.w_std),
           "Wg": mat("Wg", (d, f), cfg.w_std) if cfg.gated else None}
    if affine_noise:
        out["gamma"] = vec("gamma", d, 0.1, 1.0)
        out["beta"] = vec("beta", d, 0.1) if cfg.norm == "layernorm" else None
    else:
        out["gamma"] = np.ones(d)
        out["beta"] = np.zeros(d) if cfg.norm == "layernorm" else None
    out["b1"] = vec("b1", f, cfg.w_std) if cfg.has_bias else None
    out["bg"] = vec("bg", f, cfg.w_std) if cfg.has_bias and cfg.gated else None
    out["b2"] = vec("b2", d, cfg.w_std) if cfg.has_bias else None
    return out


def make_lora_inputs(cfg: LayerConfig, rank: int, *, affine_noise: bool = False, a_std: float = 0.05, b_std: float = 0.05) -> dict:
    """The layer's inputs plus rank-``rank`` adapters Aq, Ak, Av ~ N(0, a_std^2) [d_model, rank] and Bq, Bk, Bv ~
    N(0, b_std^2) [rank, d_q | d_kv], rounded to the storage dtype.  (Fine-tuning starts from B = 0; a non-zero B
    is drawn so that every gradient path carries signal.)"""
    out = make_inputs(cfg, affine_noise=affine_noise)
    for k, cols in (("q", cfg.d_q), ("k", cfg.d_kv), ("v", cfg.d_kv)):
        a = normal_f64(cfg.seed, TENSOR_IDS["A" + k], 0, cfg.d_model * rank).reshape(cfg.d_model, rank) * a_std
        b = normal_f64(cfg.seed, TENSOR_IDS["B" + k], 0, rank * cols).reshape(rank, cols) * b_std
        out["A" + k] = round_to_storage(a, cfg.dtype)
        out["B" + k] = round_to_storage(b, cfg.dtype)
    return out


def make_xattn_inputs(cfg, *, affine_noise: bool = False) -> dict:
    """All inputs of the cross-attention layer ``cfg`` (an ``XattnConfig``): hidden states X and output gradient dY
    [batch, seq, d_model], memory M [batch, seq_kv, d_mem] ~ N(0, 1); Wq [d_model, d_q], Wk, Wv [d_mem, d_kv],
    Wo [d_q, d_model] ~ N(0, w_std^2); vectors fp32.  Storage-rounded float64, as ``make_inputs``."""
    s = cfg.seed
    d, dm, dq, dkv = cfg.d_model, cfg.d_mem, cfg.d_q, cfg.d_kv

    def mat(name, shape, std):
        cnt = int(np.prod(shape))
        return round_to_storage(normal_f64(s, TENSOR_IDS[name], 0, cnt).reshape(shape) * std, cfg.dtype)

    def vec(name, length, std, mean=0.0):
        return (normal_f64(s, TENSOR_IDS[name], 0, length) * std + mean).astype(np.float32).astype(np.float64)

    out = {"X": mat("X", (cfg.batch, cfg.seq, d), 1.0), "dY": mat("dY", (cfg.batch, cfg.seq, d), 1.0),
           "M": mat("M", (cfg.batch, cfg.seq_kv, dm), 1.0),
           "Wq": mat("Wq", (d, dq), cfg.w_std), "Wk": mat("Wk", (dm, dkv), cfg.w_std),
           "Wv": mat("Wv", (dm, dkv), cfg.w_std), "Wo": mat("Wo", (dq, d), cfg.w_std)}
    if affine_noise:
        out["gamma"] = vec("gamma", d, 0.1, 1.0)
        out["beta"] = vec("beta", d, 0.1) if cfg.norm == "layernorm" else None
    else:
        out["gamma"] = np.ones(d)
        out["beta"] = np.zeros(d) if cfg.norm == "layernorm" else None
    for k, n in (("bq", dq), ("bk", dkv), ("bv", dkv), ("bo", d)):
        out[k] = vec(k, n, cfg.w_std) if cfg.has_bias else None
    return out
