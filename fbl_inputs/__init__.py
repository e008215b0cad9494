"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests.

This package holds the workload table and a counter-based random generator, and
none of the layer's arithmetic: no norm, no matmul, no softmax, no layout math.
"""
from .configs import CONFIGS, MLP_CONFIGS, XATTN_CONFIGS, LayerConfig, MlpConfig, XattnConfig, get_config, scaled_config
from .synth import TENSOR_IDS, make_inputs, make_lora_inputs, make_mlp_inputs, make_xattn_inputs, normal_f64, round_to_storage, to_bf16_bits

__all__ = [
    "CONFIGS", "MLP_CONFIGS", "XATTN_CONFIGS", "LayerConfig", "MlpConfig", "XattnConfig", "get_config", "scaled_config",
    "TENSOR_IDS", "make_inputs", "make_lora_inputs", "make_mlp_inputs", "make_xattn_inputs", "normal_f64", "round_to_storage", "to_bf16_bits",
]
