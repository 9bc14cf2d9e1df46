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


def check_stats(mean, invstd, ref_y, eps, mode="bf16"):
    """Batch statistics against the oracle's, at the accuracy the arithmetic predicts (not the tensors' 5e-3 bar).

    ref_y is the oracle's convolution output [..., C] (fp64).  16-bit modes: the kernels take the statistics of the
    fp16-ROUNDED output, y_i(1 + d_i) with |d_i| <= 2^-11, i.e. a rounding error of standard deviation at most
    2^-12 |y_i| per element, independent between elements.  To first order
        mean error      = (1/M) sum y_i d_i                 -> std  2^-12 sqrt(sum y_i^2) / M
        variance error  = (2/M) sum (y_i - mean) y_i d_i    -> std  2 * 2^-12 sqrt(sum (y_i - mean)^2 y_i^2) / M
        invstd, relative = variance error / (2 (var + eps)).
    The bars are SIX such standard deviations (per channel, from the oracle's own y) plus 3e-6 for the fp32 partial sums
    and the fp32 accumulators: about 3e-5 * rms at M = 2048 rows, 1e-6 at the benchmark's sizes.  A dropped 128-row tile
    moves the mean by 1e-3 * rms and more.  fp32 mode: 3e-6."""
    mean, invstd = np.asarray(mean, np.float64), np.asarray(invstd, np.float64)
    c = ref_y.shape[-1]
    y = np.asarray(ref_y, np.float64).reshape(-1, c)
    m_rows = y.shape[0]
    ref_mean = y.mean(0)
    ref_var = ((y - ref_mean) ** 2).mean(0)
    ref_invstd = 1.0 / np.sqrt(ref_var + eps)
    rms = np.sqrt(ref_mean**2 + ref_var)
    tol_mean = 3e-6 * rms
    tol_istd = np.full(c, 3e-6)
    if mode == "bf16":
        u = 2.0**-12
        tol_mean = tol_mean + 6.0 * u * np.sqrt((y * y).sum(0)) / m_rows
        tol_istd = tol_istd + 6.0 * u * np.sqrt((((y - ref_mean) * y) ** 2).sum(0)) / m_rows / (ref_var + eps)
    err_mean = np.abs(mean - ref_mean)
    err_istd = np.abs(invstd - ref_invstd) / ref_invstd
    k = int(np.argmax(err_mean / np.maximum(tol_mean, 1e-300)))
    assert (err_mean <= tol_mean).all(), f"mean[{k}]: |err| {err_mean[k]:.3e} > {tol_mean[k]:.3e} (rms {rms[k]:.3e}, {m_rows} rows)"
    k = int(np.argmax(err_istd / tol_istd))
    assert (err_istd <= tol_istd).all(), f"invstd[{k}]: relative error {err_istd[k]:.3e} > {tol_istd[k]:.3e} ({m_rows} rows)"
    return float((err_mean / np.maximum(rms, 1e-300)).max()), float(err_istd.max())
