"""Parity metrics and helpers shared by the GPU tests (no arithmetic of the method here)."""
import numpy as np

# Tolerances of the benchmark spec: bf16-in / fp32-accumulate results against the fp64 oracle, and the fp32 reference mode.
BF16_REL_L2 = 5e-3
BF16_MAX_OVER_RMS = 5e-2
F32_REL_L2 = 1e-5


def rel_l2(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = float(np.sqrt((ref * ref).sum()))
    num = float(np.sqrt(((got - ref) ** 2).sum()))
    return num / den if den > 0 else num


def max_over_rms(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt((ref * ref).mean()))
    err = float(np.abs(got - ref).max())
    return err / rms if rms > 0 else err


def check(name, got, ref, mode="bf16", report=None):
    """Assert the benchmark spec's tolerance for one tensor; returns (rel_l2, max/rms)."""
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    r, m = rel_l2(got, ref), max_over_rms(got, ref)
    if report is not None:
        report[name] = (r, m)
    if mode == "bf16":
        assert r <= BF16_REL_L2, f"{name}: rel L2 {r:.3e} > {BF16_REL_L2}"
        assert m <= BF16_MAX_OVER_RMS, f"{name}: max|err|/rms {m:.3e} > {BF16_MAX_OVER_RMS}"
    else:
        assert r <= F32_REL_L2, f"{name}: rel L2 {r:.3e} > {F32_REL_L2}"
    return r, m
