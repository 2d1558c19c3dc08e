"""Parity gates shared by the GPU tests (tolerances of the stated target, written out here).

bf16 inputs / fp32 accumulation: max-abs <= 2e-2 and mean-abs <= 2e-3 (the stated target), plus two
scale-free gates that keep their power when outputs are small (near-uniform softmax):
max|err| / max|ref| <= 1e-2 and mean|err| / mean|ref| <= 5e-3.  The output is rounded to bf16
(relative 2^-9 per element), which these allow for.
fp32 inputs: max|err| <= 1e-5 * max|ref| ("1e-5 relative", taken over the tensor because an
element-wise ratio is undefined at zeros).
"""
import numpy as np


def errors(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    return dict(max_abs=float(err.max()), mean_abs=float(err.mean()),
                max_rel=float(err.max() / max(np.abs(ref).max(), 1e-300)),
                mean_rel=float(err.mean() / max(np.abs(ref).mean(), 1e-300)))


def gate_ok(got, ref, dtype: str) -> bool:
    e = errors(got, ref)
    if not np.isfinite(np.asarray(got, dtype=np.float64)).all():
        return False
    if dtype == "f32":
        return e["max_rel"] <= 1e-5
    return e["max_abs"] <= 2e-2 and e["mean_abs"] <= 2e-3 and e["max_rel"] <= 1e-2 and e["mean_rel"] <= 5e-3


def assert_parity(got, ref, dtype: str, what: str = ""):
    e = errors(got, ref)
    assert gate_ok(got, ref, dtype), f"{what}: parity gate failed {e}"
    return e
