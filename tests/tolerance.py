"""Element-wise comparison rule used by every parity test: |got - ref| <= atol + rtol*|ref|."""
import numpy as np

# Bounds stated for this path: O and LSE 1e-2 + 1e-2|ref|; dQ, dK, dV 2e-2 + 2e-2|ref|.
FWD_ATOL = FWD_RTOL = 1e-2
BWD_ATOL = BWD_RTOL = 2e-2
# Informational-turned-enforced relative RMS bounds (the absolute terms above are weak where the
# reference is small, e.g. late rows of O or gradients under a 1e-2 upstream gradient).
FWD_REL_RMS = 5e-3
BWD_REL_RMS = 1e-2


def max_violation(got, ref, atol, rtol):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), "non-finite values in result"
    err = np.abs(got - ref)
    bound = atol + rtol * np.abs(ref)
    return float((err - bound).max()), float(err.max())


def rel_rms(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = float(np.sqrt((ref * ref).sum()))
    num = float(np.sqrt(((got - ref) ** 2).sum()))
    return num / den if den > 0 else num


def assert_close(got, ref, atol, rtol, name="", rms_bound=None):
    viol, maxerr = max_violation(got, ref, atol, rtol)
    assert viol <= 0.0, f"{name}: max|err|={maxerr:.3e} exceeds {atol}+{rtol}|ref| by {viol:.3e}"
    if rms_bound is not None:
        r = rel_rms(got, ref)
        assert r <= rms_bound, f"{name}: relative RMS error {r:.3e} > {rms_bound}"
    return maxerr


def violation_stats(got, ref, atol, rtol):
    """How far a result is from the bound, as numbers to record: the count of elements with
    |got - ref| > atol + rtol*|ref| and the largest |got - ref| / (atol + rtol*|ref|)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    ratio = np.abs(got - ref) / (atol + rtol * np.abs(ref))
    return int((ratio > 1.0).sum()), float(ratio.max()), int(ratio.size)
