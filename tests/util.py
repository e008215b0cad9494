"""Shared helpers for the tests (no method arithmetic): the tolerances and how they are applied.

fp32 storage: max error relative to max(|ref_i|, rms(ref)) must stay below 1e-4.

bf16 storage with fp32 accumulation ("2e-2 relative / 1e-2 absolute").  Three criteria, all asserted:

 1. tensor scale, every tensor:  max|e| <= 1e-2 + 2e-2 * max|ref|.
 2. scale free, every tensor with a non-zero reference:  ||e||_F / ||ref||_F <= 1e-2  (the rounding floor of
    any bf16 implementation, tests/bf16_floor.py, sits at 3e-3 .. 6e-3).
 3. element-wise, |e_i| <= 1e-2 + 2e-2 |ref_i|: the fraction of elements outside it is capped relative to the
    same fraction of the rounding floor, computed for the very layer under test from the oracle alone:
       Y, dX, dM (token tensors):       at most 10 x the floor's fraction (zero where the floor has none);
       dW*, db*, dgamma, dbeta:         at most 2 x the floor's fraction + 1e-3.  These are sums over thousands
                                        of tokens with cancellation, so their small elements carry noise in
                                        proportion to the tensor's scale in any bf16-operand implementation
                                        (floor: up to 10 % of elements at 4096 tokens); a cap tied to that floor
                                        still catches an error confined to the small elements.

 dbk is identically zero in exact arithmetic (a shift of every key leaves softmax unchanged); what an
 implementation returns is the rounding noise of bf16 dS summed over tokens and the heads of a group.  It is
 judged against max(1e-2, 2 x the floor's own max|dbk|): the stated absolute bound wherever the floor leaves
 room for it, and twice the floor where even exact sums of rounded operands exceed it.
"""
import json
import os

import numpy as np

FP32_REL = 1e-4
BF16_RTOL, BF16_ATOL = 2e-2, 1e-2
FRO_MAX = 1e-2
TOKEN_TENSORS = ("Y", "dX", "dM")
TOKEN_VIOL_OVER_FLOOR = 10.0
REDUCTION_VIOL_OVER_FLOOR, REDUCTION_VIOL_SLACK = 2.0, 1e-3
ZERO_REF = ("dbk",)


def fp32_err(got, ref):
    floor = np.sqrt(np.mean(ref ** 2)) + 1e-30
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor)))


def bf16_figures(got, ref):
    e = np.abs(got - ref)
    return dict(max_abs=float(e.max()),
                worst_over_bound=float(e.max() / (BF16_ATOL + BF16_RTOL * np.abs(ref).max())),
                fro=float(np.linalg.norm(got - ref) / (np.linalg.norm(ref) + 1e-300)),
                viol=float((e > BF16_ATOL + BF16_RTOL * np.abs(ref)).mean()),
                numel=int(ref.size))


def bf16_ok(name, got, ref, floor=None, zero_ref_names=ZERO_REF):
    """Apply the criteria above.  ``floor``: this tensor's entry of bf16_floor.floor_figures for the same layer;
    None (intermediates, which the floor does not list) applies criteria 1 and 2 only.  ``zero_ref_names``: tensors
    whose reference is identically zero (dbk, unless a rotary embedding sits between the key projection and the scores).
    Returns (ok, figures, list of failed criteria)."""
    f = bf16_figures(got, ref)
    failed = []
    if name not in zero_ref_names and np.abs(ref).max() < 1e-9:
        # a reference that vanishes identically (one token per sequence: dS = 0, hence dQ, dK, dWq, dWk, dbq):
        # only the absolute part of the bound means anything
        if f["max_abs"] > BF16_ATOL:
            failed.append("zero-reference bound")
        return not failed, f, failed
    if name in zero_ref_names:
        bound = max(BF16_ATOL, 2.0 * floor["max_abs"]) if floor is not None else BF16_ATOL
        f["worst_over_bound"] = f["max_abs"] / bound
        if f["max_abs"] > bound:
            failed.append("zero-reference bound")
        return not failed, f, failed
    if f["worst_over_bound"] > 1.0:
        failed.append("tensor-scale bound")
    if f["fro"] > FRO_MAX:
        failed.append("Frobenius bound")
    if floor is not None:
        if name in TOKEN_TENSORS:
            cap = TOKEN_VIOL_OVER_FLOOR * floor["viol"]
        else:
            cap = REDUCTION_VIOL_OVER_FLOOR * floor["viol"] + REDUCTION_VIOL_SLACK
        f["viol_cap"] = cap
        if f["viol"] > cap:
            failed.append("element-wise violating fraction")
    return not failed, f, failed


def report(name, f, floor=None):
    s = (f"{name:7s} max|e|={f['max_abs']:.3e} worst/bound={f['worst_over_bound']:.3f} fro={f['fro']:.3e} "
         f"elementwise-viol={f['viol']:.2e}")
    if floor is not None:
        s += f" | floor: worst/bound={floor['worst_over_bound']:.3f} fro={floor['fro']:.3e} viol={floor['viol']:.2e}"
    return s


def record(case, figures, floors):
    """Append one layer's figures to the JSON-lines file named by FBL_PARITY_REPORT (if set)."""
    path = os.environ.get("FBL_PARITY_REPORT")
    if path:
        with open(path, "a") as fh:
            fh.write(json.dumps({"case": case, "gpu": figures, "floor": floors}) + "\n")
