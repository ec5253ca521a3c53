"""Shared helpers of the GPU parity tests: tolerances and comparison metrics.

Tolerances (from the benchmark's statement of the task):
  * pos masks and positive counts: bit-exact / equal integers;
  * the two local and two global means: relative error <= 1e-6;
  * updated w and err: <= 1e-5 in the normalised metric below.

Metric for w and err.  The residual e' = v - g_hat cancels to ~0 wherever v is
close to a mean, so a strict element-wise relative error is unbounded even for
perfect fp32 arithmetic.  The error is therefore normalised by
max(|reference_i|, tau) with tau_err = max(m_pos, m_neg) (the scale of v and
g_hat that were subtracted) and tau_w = RMS(w_reference).
"""
import numpy as np

MEANS_RTOL = 1e-6
STATE_TOL = 1e-5


def rel_err_means(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    denom = np.where(ref != 0, np.abs(ref), 1.0)
    return float(np.max(np.abs(got - ref) / denom)) if got.size else 0.0


def normalised_err(got, ref, tau):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    tau = max(float(tau), 1e-30)
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), tau))) if got.size else 0.0


def tau_err(global_means):
    return float(max(abs(float(global_means[0])), abs(float(global_means[1]))))


def tau_w(w_ref):
    w = np.asarray(w_ref, np.float64)
    return float(np.sqrt(np.mean(w * w))) if w.size else 1.0


def assert_means(got, ref, what="means"):
    err = rel_err_means(got, ref)
    assert err <= MEANS_RTOL, f"{what}: relative error {err:.3e} > {MEANS_RTOL}"


def count_outliers(got, ref, tau, tol=STATE_TOL):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    tau = max(float(tau), 1e-30)
    return int(np.count_nonzero(np.abs(got - ref) > tol * np.maximum(np.abs(ref), tau)))


def assert_state(w_got, w_ref, e_got, e_ref, gm_ref, what="", max_outliers=0):
    """``max_outliers`` > 0 only in free-running multi-step comparisons, where an element
    whose compensated value sits at rounding level may legitimately change group."""
    bad = count_outliers(w_got, w_ref, tau_w(w_ref))
    assert bad <= max_outliers, (f"{what} w: {bad} elements over {STATE_TOL} "
                                 f"(max normalised error {normalised_err(w_got, w_ref, tau_w(w_ref)):.3e})")
    if e_got is not None:
        bad = count_outliers(e_got, e_ref, tau_err(gm_ref))
        assert bad <= max_outliers, (f"{what} err: {bad} elements over {STATE_TOL} "
                                     f"(max normalised error {normalised_err(e_got, e_ref, tau_err(gm_ref)):.3e})")
