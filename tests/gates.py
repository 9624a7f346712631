"""Pass/fail gates shared by the parity tests.

stated gate : |err| <= 1e-2 + 1e-2 * |ref|                       (the contract)
tight gate  : |err| <= 2^-7 * (|ref| + rms_row(ref))             (what a correct fp32-accumulate,
              bf16-output kernel meets with margin: output rounding is 2^-9 |ref|, rounding the
              probabilities to bf16 for the tensor-core PV product adds < 2^-9 of the row rms)

With N(0,1) data the outputs of long sequences have rms ~ sqrt(e / L) (0.009 at L = 32768), below
the absolute term of the stated gate, so the stated gate alone cannot see a dropped chunk; the
tight gate can.
"""
import numpy as np


def stated_violations(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    bad = ~(np.abs(got - ref) <= 1e-2 + 1e-2 * np.abs(ref))
    return int(bad.sum())


def tight_violations(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    bad = ~(np.abs(got - ref) <= 2.0 ** -7 * (np.abs(ref) + rms))
    return int(bad.sum())


def tight_ratio(got, ref):
    """max over elements of |err| / tight bound (<= 1 passes)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    bound = 2.0 ** -7 * (np.abs(ref) + rms)
    with np.errstate(divide="ignore", invalid="ignore"):
        r = np.where(bound > 0, np.abs(got - ref) / bound, np.where(got == ref, 0.0, np.inf))
    return float(np.nanmax(r)) if r.size else 0.0
