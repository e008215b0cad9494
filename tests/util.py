"""Shared helpers for the tests (no method arithmetic)."""
import numpy as np

# Tolerances.  fp32 storage: max error relative to max(|ref_i|, rms(ref)) must stay below 1e-4.
# bf16 storage with fp32 accumulation: |e| <= 1e-2 + 2e-2 |ref| element by element for the token
# tensors Y and dX; for the token-axis reductions (dW, db, dgamma, dbeta), whose small elements carry
# rounding noise proportional to the tensor's scale, the same bound with |ref| taken as max|ref|.
FP32_REL = 1e-4
BF16_RTOL, BF16_ATOL = 2e-2, 1e-2
ELEMENTWISE = ("Y", "dX")


def fp32_err(got, ref):
    floor = np.sqrt(np.mean(ref ** 2)) + 1e-30
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor)))


def bf16_ok(name, got, ref):
    e = np.abs(got - ref)
    if name in ELEMENTWISE:
        bound = BF16_ATOL + BF16_RTOL * np.abs(ref)
        return bool((e <= bound).all()), float((e / bound).max())
    bound = BF16_ATOL + BF16_RTOL * np.abs(ref).max()
    return bool(e.max() <= bound), float(e.max() / bound)


def report(name, got, ref):
    e = np.abs(got - ref)
    mx = np.abs(ref).max() + 1e-30
    viol = float((e > BF16_ATOL + BF16_RTOL * np.abs(ref)).mean())
    return (f"{name:7s} max|e|={e.max():.3e} max|e|/max|ref|={e.max() / mx:.3e} "
            f"fro={np.linalg.norm(got - ref) / (np.linalg.norm(ref) + 1e-30):.3e} elementwise-viol={viol:.2e}")
