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


# ---------------------------------------------------------------- helpers for the full-size comparisons
def strict_rel_err(got, ref):
    """Plain element-wise relative error max_i |got - ref| / |ref| (elements with ref == 0 skipped).
    Reported for information next to the normalised metric: it is unbounded by construction for the
    residual (see the module docstring), so nothing is asserted on it."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    nz = ref != 0
    return float(np.max(np.abs(got[nz] - ref[nz]) / np.abs(ref[nz]))) if nz.any() else 0.0


def oracle_encode_by_worker(oracle, g, e, mode, want_mask=False, threads=None):
    """oracle.encode called once per worker, the P calls running side by side on host threads
    (ctypes releases the interpreter lock).  Every call is the unmodified oracle on one worker's
    whole vector, so each result is exactly what a single call over all workers returns."""
    from concurrent.futures import ThreadPoolExecutor
    P = g.shape[0]

    def one(p):
        return oracle.encode(g[p:p + 1], e[p:p + 1] if e is not None else None, mode=mode, want_mask=want_mask)

    with ThreadPoolExecutor(max_workers=threads or P) as pool:
        parts = list(pool.map(one, range(P)))
    lm = np.concatenate([x[0] for x in parts])
    cnt = np.concatenate([x[1] for x in parts])
    mask = np.concatenate([x[2] for x in parts]) if want_mask else None
    return lm, cnt, mask


def oracle_decode_by_chunks(oracle, w, g, e, lm, gm, lr, mode, chunks=16, mom=None, beta=0.0, wd=0.0):
    """oracle.decode_update (or its momentum form) over the whole vector as ``chunks`` calls on
    consecutive element ranges, side by side on host threads.  The decode of one element depends
    only on that element and on the means, so the chunked calls give, element by element, the
    results of one call; the oracle itself is untouched."""
    from concurrent.futures import ThreadPoolExecutor
    n = g.shape[1]
    bounds = np.linspace(0, n, min(chunks, n) + 1).astype(np.int64)

    def one(k):
        lo, hi = int(bounds[k]), int(bounds[k + 1])
        if hi <= lo:
            return
        wk = w[..., lo:hi]
        ek = e[:, lo:hi] if e is not None else None
        if mom is None:
            oracle.decode_update(wk, g[:, lo:hi], ek, lm, gm, lr, mode=mode)
        else:
            oracle.decode_update_momentum(wk, mom[..., lo:hi], g[:, lo:hi], ek, lm, gm, lr, beta, wd, mode=mode)

    with ThreadPoolExecutor(max_workers=len(bounds) - 1) as pool:
        list(pool.map(one, range(len(bounds) - 1)))


def device_outliers(got_dev, ref_host, tau, tol=STATE_TOL, chunk=1 << 27):
    """count_outliers and the largest normalised error with the arithmetic of the comparison done
    on the GPU (the reference is uploaded chunk by chunk): plumbing for arrays of 10^9 elements."""
    import torch
    tau = max(float(tau), 1e-30)
    got = got_dev.reshape(-1) if got_dev.is_contiguous() else None
    ref_flat = ref_host.reshape(-1)
    bad, worst = 0, 0.0
    n = ref_flat.shape[0]
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        r = torch.from_numpy(ref_flat[lo:hi]).to(got_dev.device, non_blocking=False).double()
        x = (got[lo:hi] if got is not None else got_dev.reshape(-1)[lo:hi]).double()
        rel = (x - r).abs() / torch.clamp(r.abs(), min=tau)
        bad += int((rel > tol).sum().item())
        worst = max(worst, float(rel.max().item()))
    return bad, worst
