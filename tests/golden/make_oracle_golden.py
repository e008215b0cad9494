"""Writes tests/golden/oracle_layer_tiny.txt: values of the float64 oracle on two tiny seeded layers.

Run from the repository root:  python tests/golden/make_oracle_golden.py

The file is a drift guard, not a pin to the paper: the pins in tests/test_oracle_pins.py fix the oracle to what the
mathematics determines; this fixture makes any later change of its arithmetic (intended or not) show up as a diff
that has to be committed together with its justification.  Only oracle/ and the seeded input generator are used.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from fbl_inputs import LayerConfig, make_inputs  # noqa: E402
from oracle import layer as orc  # noqa: E402

CASES = {
    # layer norm, causal, grouped-query (4 query / 2 KV heads), biases and residual
    "ln_causal_gqa": LayerConfig("g1", 2, 7, 12, 4, 2, 3, "fp32", "layernorm", True, True, True, 1e-5, 101, 0.3),
    # RMS norm, full attention, multi-head, no bias, no residual
    "rms_full_mha": LayerConfig("g2", 1, 5, 8, 2, 2, 4, "fp32", "rmsnorm", False, False, False, 1e-6, 102, 0.3),
}
NAMES = ("Y", "dX", "dWq", "dWk", "dWv", "dWo", "dgamma")


def values(cfg):
    Y, saved, g = orc.layer_fwd_bwd(cfg, make_inputs(cfg, affine_noise=True))
    out = {"Y": Y}
    out.update({n: g[n] for n in NAMES[1:]})
    return out


def lines():
    for key, cfg in CASES.items():
        v = values(cfg)
        for n in NAMES:
            a = np.asarray(v[n], dtype=np.float64).ravel()
            # the sum, the sum of squares and three fixed elements of every tensor
            picks = [a[0], a[a.size // 2], a[-1]]
            yield "%s %s %d %.17e %.17e %s" % (key, n, a.size, a.sum(), (a * a).sum(), " ".join("%.17e" % x for x in picks))


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_layer_tiny.txt")
    with open(path, "w") as f:
        f.write("# case tensor size sum sum_of_squares first middle last   (float64 oracle; see make_oracle_golden.py)\n")
        for ln in lines():
            f.write(ln + "\n")
    print("wrote", path)
