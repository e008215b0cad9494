"""Shared helpers for the tests (no method arithmetic)."""
import numpy as np

# Tolerances.
# fp32 storage: max error relative to max(|ref_i|, rms(ref)) must stay below 1e-4.
# bf16 storage with fp32 accumulation ("2e-2 relative / 1e-2 absolute"): per tensor, max|e| must not exceed
# 1e-2 + 2e-2 * max|ref|.  For the token tensors Y and dX the element-wise form |e| <= 1e-2 + 2e-2 |ref| must
# also hold for all but a 1e-5 fraction of elements: isolated elements can miss it by a few per cent because the
# bf16 rounding of intermediates of magnitude ~4 (ulp 0.03) lands on outputs of magnitude < 1.  The token-axis
# reductions (dW, db, dgamma, dbeta) are judged on the tensor scale only: their small elements carry rounding
# noise proportional to the tensor's scale in any bf16-operand implementation.  The element-wise violation
# fraction is printed for every tensor.
FP32_REL = 1e-4
BF16_RTOL, BF16_ATOL = 2e-2, 1e-2
ELEMENTWISE = ("Y", "dX")
ELEMENTWISE_MAX_VIOLATING_FRACTION = 1e-5


def fp32_err(got, ref):
    floor = np.sqrt(np.mean(ref ** 2)) + 1e-30
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor)))


def bf16_ok(name, got, ref):
    e = np.abs(got - ref)
    bound = BF16_ATOL + BF16_RTOL * np.abs(ref).max()
    ok = bool(e.max() <= bound)
    worst = float(e.max() / bound)
    if name in ELEMENTWISE:
        viol = float((e > BF16_ATOL + BF16_RTOL * np.abs(ref)).mean())
        ok = ok and viol <= ELEMENTWISE_MAX_VIOLATING_FRACTION
    return ok, worst


def report(name, got, ref):
    e = np.abs(got - ref)
    mx = np.abs(ref).max() + 1e-30
    viol = float((e > BF16_ATOL + BF16_RTOL * np.abs(ref)).mean())
    return (f"{name:7s} max|e|={e.max():.3e} max|e|/max|ref|={e.max() / mx:.3e} "
            f"fro={np.linalg.norm(got - ref) / (np.linalg.norm(ref) + 1e-30):.3e} elementwise-viol={viol:.2e}")
