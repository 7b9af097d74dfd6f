"""Shared helpers for the tests: the error metric of the parity gate and small conversions."""
import numpy as np

GOLDEN = __import__("os").path.join(__import__("os").path.dirname(__file__), "golden")

# Gate for Y, dX, dA, dB (bf16 inputs, fp32 accumulation on the GPU): max relative error 2e-2, where the
# error of element i is |got_i - ref_i| / max(|ref_i|, rms(ref)).  The RMS floor keeps elements that cancel
# to (almost) zero from blowing up the ratio; the GPU rounds W, H, G and its outputs to bf16 (2^-9 each).
REL_TOL = 2e-2


def rel_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(ref * ref)))
    denom = np.maximum(np.abs(ref), rms if rms > 0 else 1.0)
    return float(np.max(np.abs(got - ref) / denom))


def golden_lines(name):
    with open(__import__("os").path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
