"""B200-native attention-layer training step on one unified tiled layout (ctypes binding).

The shared library is built in-tree by ``paper_2607_21624_b200.build``; importing this
package never falls back to another implementation: if the library is missing or a
CUDA device is absent, calls raise.
"""
from .binding import (FblError, Plan, lib, load_library, LayerRunner, DTYPES, TENSOR, MAP, WS,
                      desc_from_config, aligned_bytes, guard_bands_intact, selftest_wait_timeout)

from .lora import LoraRunner
from .xattn import XattnRunner
from .mlp import MlpPlan, MlpRunner, mlp_desc_from_config, MLP_TENSOR, MLP_WS

__all__ = ["LoraRunner", "XattnRunner", "MlpPlan", "MlpRunner", "mlp_desc_from_config", "MLP_TENSOR", "MLP_WS",
           "FblError", "Plan", "lib", "load_library", "LayerRunner", "DTYPES", "TENSOR", "MAP", "WS",
           "desc_from_config", "aligned_bytes", "guard_bands_intact", "selftest_wait_timeout"]
