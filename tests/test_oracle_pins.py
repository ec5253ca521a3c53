"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself — hand-worked fixtures, exact rational brute force written
straight from the definitions, library reductions, closed forms and invariants
that the paper's Section 3.1, Algorithm 1 and Eq. 13 fix."""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
EF, ALG1 = oracle.MODE_EF, oracle.MODE_ALG1


def _load(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def _f32(rows):
    return np.array([[float(x) for x in r] for r in rows], np.float32)


# ---------------------------------------------------------------- hand-worked fixtures
def test_golden_e1_error_feedback_two_steps():
    fx = _load("e1_ef_single_worker_two_steps.json")
    w = np.array(fx["w0"], np.float32)
    e = _f32(fx["e0"])
    for st in fx["steps"]:
        g = _f32(st["g"])
        lm, cnt, mask = oracle.encode(g, e, mode=EF, want_mask=True)
        assert lm.tolist() == st["local_means"]
        assert cnt.tolist() == st["pos_counts"]
        assert mask.tolist() == st["mask_words"]
        assert oracle.global_average(lm).tolist() == st["global_means"]
        lm2, gm2, cnt2 = oracle.step(w, g, e, fx["lr"], mode=EF)
        assert lm2.tolist() == st["local_means"] and gm2.tolist() == st["global_means"]
        assert e.tolist() == st["e"]
        assert w.tolist() == st["w"]


@pytest.mark.parametrize("mode_name", ["EF", "ALG1"])
def test_golden_e2_two_workers(mode_name):
    fx = _load("e2_two_workers.json")
    mode = EF if mode_name == "EF" else ALG1
    g = _f32(fx["g"])
    e = np.zeros_like(g)
    lm, cnt, mask = oracle.encode(g, e if mode == EF else None, mode=mode, want_mask=True)
    assert lm.tolist() == fx["local_means"]
    assert cnt.tolist() == fx["pos_counts"]
    assert mask.tolist() == fx["mask_words"]
    gm = oracle.global_average(lm)
    assert gm.tolist() == fx["global_means"]
    # replicated w, lr = 1, w0 = 0  =>  w^p = -g_hat^p
    w_rep = np.zeros_like(g)
    e_rep = e.copy()
    oracle.decode_update(w_rep, g, e_rep, lm, gm, fx["lr"], mode=mode)
    assert (-w_rep).tolist() == fx[mode_name]["g_hat"]
    assert e_rep.tolist() == fx[mode_name]["e" if mode == EF else "eps"]
    # one shared w  =>  w = -mean_p g_hat^p
    w_sh = np.array(fx["w0"], np.float32)
    e_sh = e.copy()
    oracle.decode_update(w_sh, g, e_sh, lm, gm, fx["lr"], mode=mode)
    assert (-w_sh).tolist() == fx[mode_name]["mean_g_hat"]
    assert e_sh.tolist() == e_rep.tolist()


def test_golden_e3_empty_group_and_signed_zero():
    fx = _load("e3_empty_group_signed_zero.json")
    g = _f32(fx["g"])
    assert np.signbit(g[0, 4])  # the fixture really holds -0.0
    lm, cnt, mask = oracle.encode(g, None, mode=ALG1, want_mask=True)
    assert cnt.tolist() == fx["pos_counts"]
    assert mask.tolist() == fx["mask_words"]
    assert lm[0, 0] == np.float32(1.2) and lm[0, 1] == 0.0
    # all-negative vector: the positive group is the empty one
    lm, cnt, _ = oracle.encode(_f32([[-1, -2, -6]]), None, mode=ALG1)
    assert lm.tolist() == [[0.0, 3.0]] and cnt.tolist() == [0]


# ---------------------------------------------------------------- exact rational brute force
def _brute_means(v):
    """Section 3.1 in exact rationals: mean of the entries >= 0, mean of |entries < 0|."""
    pos = [Fraction(float(x)) for x in v if x >= 0]
    neg = [-Fraction(float(x)) for x in v if x < 0]
    mu_pos = sum(pos, Fraction(0)) / len(pos) if pos else Fraction(0)
    mu_neg = sum(neg, Fraction(0)) / len(neg) if neg else Fraction(0)
    return mu_pos, mu_neg, len(pos)


def _round32(fr: Fraction) -> float:
    # Fraction -> nearest double (correctly rounded by Python) -> nearest float; the double
    # rounding can differ from direct rounding by at most one fp32 ulp in rare ties.
    return float(np.float32(float(fr)))


def _ulp_close(a, b, ulps=1):
    a, b = np.float32(a), np.float32(b)
    return abs(float(a) - float(b)) <= ulps * float(np.spacing(max(abs(a), abs(b), np.float32(1e-45))))


@pytest.mark.parametrize("seed", range(40))
def test_bruteforce_rational_small_n(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 17))
    P = int(rng.integers(1, 5))
    g = (rng.standard_normal((P, n)) * 10.0 ** rng.uniform(-4, 1)).astype(np.float32)
    e = (rng.standard_normal((P, n)) * 10.0 ** rng.uniform(-4, 1)).astype(np.float32)
    if seed % 3 == 0:
        g[rng.random((P, n)) < 0.3] = 0.0
        e[g == 0.0] = 0.0
    lr = 0.25
    for mode in (EF, ALG1):
        v = (g + e).astype(np.float32) if mode == EF else g
        lm, cnt, mask = oracle.encode(g, e if mode == EF else None, mode=mode, want_mask=True)
        exact = [_brute_means(v[p]) for p in range(P)]
        for p in range(P):
            assert _ulp_close(lm[p, 0], _round32(exact[p][0]))
            assert _ulp_close(lm[p, 1], _round32(exact[p][1]))
            assert int(cnt[p]) == exact[p][2]
            bits = sum(1 << i for i in range(n) if v[p, i] >= 0)
            assert int(mask[p, 0]) == bits
        # global means: unweighted average of the fp32 local means, exactly
        gm = oracle.global_average(lm)
        for k in range(2):
            ex = sum((Fraction(float(lm[p, k])) for p in range(P)), Fraction(0)) / P
            assert _ulp_close(gm[k], _round32(ex))
        # decode + update against exact rationals, replicated and shared w
        w0 = rng.standard_normal(n).astype(np.float32)
        m_pos, m_neg = Fraction(float(gm[0])), Fraction(float(gm[1]))
        ghat = [[None] * n for _ in range(P)]
        resid = [[None] * n for _ in range(P)]
        for p in range(P):
            for i in range(n):
                vi = Fraction(float(v[p, i]))
                mean_vec = m_pos if v[p, i] >= 0 else -m_neg
                if mode == EF:
                    ghat[p][i] = mean_vec
                    resid[p][i] = vi - mean_vec
                else:
                    enc = Fraction(float(lm[p, 0])) if v[p, i] >= 0 else -Fraction(float(lm[p, 1]))
                    resid[p][i] = vi - enc
                    ghat[p][i] = vi - enc + mean_vec
        w_rep = np.tile(w0, (P, 1))
        e_rep = e.copy()
        oracle.decode_update(w_rep, g, e_rep, lm, gm, lr, mode=mode)
        w_sh = w0.copy()
        e_sh = e.copy()
        oracle.decode_update(w_sh, g, e_sh, lm, gm, lr, mode=mode)
        lr_fr = Fraction(float(np.float32(lr)))
        for i in range(n):
            mean_g = sum((ghat[p][i] for p in range(P)), Fraction(0)) / P
            assert _ulp_close(w_sh[i], _round32(Fraction(float(w0[i])) - lr_fr * mean_g))
            for p in range(P):
                assert _ulp_close(w_rep[p, i], _round32(Fraction(float(w0[i])) - lr_fr * ghat[p][i]))
                assert _ulp_close(e_rep[p, i], _round32(resid[p][i]))
        assert np.array_equal(e_sh, e_rep)


def test_all_sign_patterns_n4():
    """Every one of the 3**4 sign patterns (negative / zero / positive) of a length-4 vector."""
    vals = {-1: -3.0, 0: 0.0, 1: 5.0}
    for code in range(3 ** 4):
        signs = [(code // 3 ** k) % 3 - 1 for k in range(4)]
        v = np.array([[vals[s] * (k + 1) for k, s in enumerate(signs)]], np.float32)
        lm, cnt, mask = oracle.encode(v, None, mode=ALG1, want_mask=True)
        mu_pos, mu_neg, n_pos = _brute_means(v[0])
        assert lm[0, 0] == _round32(mu_pos) and lm[0, 1] == _round32(mu_neg)
        assert int(cnt[0]) == n_pos == sum(s >= 0 for s in signs)
        assert int(mask[0, 0]) == sum(1 << k for k, s in enumerate(signs) if s >= 0)


# ---------------------------------------------------------------- library reductions and statistics
@pytest.mark.parametrize("n", [1, 31, 32, 33, 1000, 100003])
def test_means_match_numpy_masked_mean(n):
    rng = np.random.default_rng(n)
    g = (rng.standard_normal((3, n)) * 1e-3).astype(np.float32)
    e = (rng.standard_normal((3, n)) * 1e-4).astype(np.float32)
    v = (g + e).astype(np.float32)
    lm, cnt, mask = oracle.encode(g, e, mode=EF, want_mask=True)
    for p in range(3):
        vp = v[p].astype(np.float64)
        mu_pos = vp[vp >= 0].mean() if (vp >= 0).any() else 0.0
        mu_neg = (-vp[vp < 0]).mean() if (vp < 0).any() else 0.0
        assert lm[p, 0] == pytest.approx(mu_pos, rel=2e-7, abs=0)
        assert lm[p, 1] == pytest.approx(mu_neg, rel=2e-7, abs=0)
        assert int(cnt[p]) == int((vp >= 0).sum())
        packed = np.packbits((vp >= 0).astype(np.uint8), bitorder="little")
        packed = np.pad(packed, (0, (-len(packed)) % 4)).view(np.uint32)
        assert np.array_equal(mask[p], packed)


def test_half_normal_and_laplace_means():
    """Zero-centred normal gradients (the paper's Fig. 1 observation): both group means
    approach sigma*sqrt(2/pi); Laplace(0, b): both approach b."""
    rng = np.random.default_rng(7)
    n = 1 << 20
    sigma = 1e-3
    g = (rng.standard_normal((1, n)) * sigma).astype(np.float32)
    lm, cnt, _ = oracle.encode(g, None, mode=ALG1)
    expect = sigma * math.sqrt(2.0 / math.pi)
    assert lm[0, 0] == pytest.approx(expect, rel=5e-3)
    assert lm[0, 1] == pytest.approx(expect, rel=5e-3)
    assert abs(int(cnt[0]) - n / 2) < 4 * math.sqrt(n) / 2
    b = 3e-4
    g = rng.laplace(0.0, b, (1, n)).astype(np.float32)
    lm, _, _ = oracle.encode(g, None, mode=ALG1)
    assert lm[0, 0] == pytest.approx(b, rel=5e-3) and lm[0, 1] == pytest.approx(b, rel=5e-3)


# ---------------------------------------------------------------- invariants of Eq. 2
def _enc(v, lm):
    return np.where(v >= 0, np.float64(lm[0]), -np.float64(lm[1]))


def test_enc_preserves_group_sums_and_is_idempotent():
    rng = np.random.default_rng(11)
    v = rng.integers(-50, 50, (1, 4096)).astype(np.float32)  # integers: sums are exact
    lm, cnt, _ = oracle.encode(v, None, mode=ALG1)
    enc = _enc(v[0], lm[0])
    pos = v[0] >= 0
    assert enc[pos].sum() == pytest.approx(v[0][pos].astype(np.float64).sum(), rel=1e-6)
    assert enc[~pos].sum() == pytest.approx(v[0][~pos].astype(np.float64).sum(), rel=1e-6)
    lm2, cnt2, _ = oracle.encode(enc.astype(np.float32)[None, :], None, mode=ALG1)
    assert np.array_equal(lm2, lm) and np.array_equal(cnt2, cnt)


def test_scale_by_power_of_two_is_bit_exact_and_negation_swaps_groups():
    rng = np.random.default_rng(12)
    v = (rng.standard_normal((2, 5000))).astype(np.float32)
    v[v == 0] = 1.0
    lm, cnt, mask = oracle.encode(v, None, mode=ALG1, want_mask=True)
    lm8, cnt8, mask8 = oracle.encode(v * np.float32(8.0), None, mode=ALG1, want_mask=True)
    assert np.array_equal(lm8, lm * np.float32(8.0))
    assert np.array_equal(cnt8, cnt) and np.array_equal(mask8, mask)
    lmn, cntn, _ = oracle.encode(-v, None, mode=ALG1)
    assert np.array_equal(lmn, lm[:, ::-1])
    assert np.array_equal(cntn, 5000 - cnt)


# ---------------------------------------------------------------- global average
def test_global_average_special_cases():
    lm = np.array([[0.375, 1.5]], np.float32)
    assert oracle.global_average(lm).tolist() == [0.375, 1.5]           # P = 1: m = mu
    lm = np.tile(np.array([[0.1, 0.7]], np.float32), (5, 1))
    assert np.array_equal(oracle.global_average(lm), lm[0])             # identical workers
    rng = np.random.default_rng(3)
    lm = rng.random((7, 2)).astype(np.float32)
    a = oracle.global_average(lm)
    b = oracle.global_average(lm[rng.permutation(7)])
    assert np.allclose(a, b, rtol=1e-7, atol=0)
    assert a[0] == pytest.approx(lm[:, 0].astype(np.float64).mean(), rel=1e-7)
    # an empty group's 0 still counts in the divide-by-P (Allreduce average divides by P)
    assert oracle.global_average(np.array([[2, 0], [4, 6]], np.float32)).tolist() == [3.0, 3.0]


# ---------------------------------------------------------------- error-feedback identities
def _random_state(seed, P, n):
    rng = np.random.default_rng(seed)
    g = (rng.standard_normal((P, n)) * 1e-3).astype(np.float32)
    e = (rng.standard_normal((P, n)) * 3e-4).astype(np.float32)
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    return g, e, w


@pytest.mark.parametrize("P", [1, 2, 4])
def test_error_feedback_identity_and_group_sums(P):
    n = 20000
    g, e, w = _random_state(100 + P, P, n)
    v = (g + e).astype(np.float32)
    e_new = e.copy()
    lm, gm, cnt = oracle.step(w, g, e_new, 0.1, mode=EF)
    ghat = np.where(v >= 0, gm[0], -gm[1]).astype(np.float64)
    # err_new + g_hat == g + err_old, element-wise
    lhs = e_new.astype(np.float64) + ghat
    assert np.max(np.abs(lhs - v.astype(np.float64))) <= 2 * np.spacing(np.float32(np.abs(v).max()))
    # per worker: sum of the residual over the positive group = n_pos * (mu_pos^p - m_pos)
    for p in range(P):
        pos = v[p] >= 0
        s = e_new[p][pos].astype(np.float64).sum()
        assert s == pytest.approx(int(cnt[p]) * (float(lm[p, 0]) - float(gm[0])), abs=1e-6 * n * 1e-3)
        s = e_new[p][~pos].astype(np.float64).sum()
        assert s == pytest.approx(-(n - int(cnt[p])) * (float(lm[p, 1]) - float(gm[1])), abs=1e-6 * n * 1e-3)


def test_two_valued_input_leaves_no_residual_single_worker():
    v = np.where(np.arange(1000) % 3 == 0, 0.75, -0.125).astype(np.float32)[None, :]
    e = np.zeros_like(v)
    w = np.zeros(1000, np.float32)
    oracle.step(w, v, e, 1.0, mode=EF)
    assert not e.any()
    assert np.array_equal(-w, v[0])


# ---------------------------------------------------------------- Algorithm 1 literal mode
def test_alg1_single_worker_is_dense_sgd():
    """P = 1: the global means equal the local ones, so Algorithm 1 hands back g itself and
    the update is the plain axpy w <- w - lr*g."""
    n = 50000
    g, _, w = _random_state(5, 1, n)
    w_ref = (w.astype(np.float64) - np.float64(np.float32(0.1)) * g[0].astype(np.float64))
    oracle.step(w, g, None, 0.1, mode=ALG1)
    assert np.max(np.abs(w.astype(np.float64) - w_ref)) <= 1.01 * np.spacing(np.abs(w).max())


def test_alg1_matches_eq13_closed_form():
    P, n, lr = 4, 30000, 0.05
    g, _, w0 = _random_state(6, P, n)
    eps = np.zeros_like(g)
    w = np.tile(w0, (P, 1))
    lm, gm, _ = oracle.step(w, g, eps, lr, mode=ALG1)
    for p in range(P):
        gp = g[p].astype(np.float64)
        enc = _enc(g[p], lm[p])
        mean_vec = np.where(g[p] >= 0, np.float64(gm[0]), -np.float64(gm[1]))
        ghat = gp + (mean_vec - enc)                       # Eq. 13: g + (mean vector - enc(g))
        ref = w0.astype(np.float64) - np.float64(np.float32(lr)) * ghat
        assert np.max(np.abs(w[p] - ref)) <= 1.01 * np.spacing(np.abs(w0).max())
        assert np.max(np.abs(eps[p] - (gp - enc))) <= np.spacing(np.float32(np.abs(g).max()))
    # identical workers: every local mean equals the global one, so g_hat = g
    g_same = np.tile(g[:1], (P, 1))
    w2 = np.tile(w0, (P, 1))
    oracle.step(w2, g_same, None, lr, mode=ALG1)
    ref = w0.astype(np.float64) - np.float64(np.float32(lr)) * g[0].astype(np.float64)
    assert np.max(np.abs(w2 - ref[None, :])) <= 1.01 * np.spacing(np.abs(w0).max())


# ---------------------------------------------------------------- weight layouts, payload, strides
@pytest.mark.parametrize("mode", [EF, ALG1])
def test_shared_w_is_mean_of_replicas_and_closed_form(mode):
    P, n, lr = 3, 10000, 0.2
    g, e, w0 = _random_state(8, P, n)
    e1, e2 = e.copy(), e.copy()
    w_rep = np.tile(w0, (P, 1))
    lm, gm, _ = oracle.step(w_rep, g, e1, lr, mode=mode)
    w_sh = w0.copy()
    oracle.step(w_sh, g, e2, lr, mode=mode)
    assert np.array_equal(e1, e2)
    assert np.max(np.abs(w_sh - w_rep.astype(np.float64).mean(axis=0))) <= 2 * np.spacing(np.abs(w0).max())
    if mode == EF:  # w_i <- w_i - (lr/P) (k_i m_pos - (P - k_i) m_neg), k_i = #workers with v >= 0
        k = ((g + e).astype(np.float32) >= 0).sum(axis=0)
        ref = w0.astype(np.float64) - np.float64(np.float32(lr)) / P * (k * float(gm[0]) - (P - k) * float(gm[1]))
        assert np.max(np.abs(w_sh - ref)) <= 1.01 * np.spacing(np.abs(w0).max())


def test_payload_is_two_floats_per_worker_and_strides_are_honoured():
    P, n, pad = 3, 777, 5
    rng = np.random.default_rng(9)
    big_g = np.full((P, n + pad), np.nan, np.float32)
    big_e = np.full((P, n + pad), np.nan, np.float32)
    big_g[:, :n] = rng.standard_normal((P, n))
    big_e[:, :n] = rng.standard_normal((P, n)) * 0.1
    lm, cnt, _ = oracle.encode(big_g[:, :n], big_e[:, :n], mode=EF)
    assert lm.shape == (P, 2) and lm.dtype == np.float32      # 64 bits per worker
    lm_c, cnt_c, _ = oracle.encode(np.ascontiguousarray(big_g[:, :n]), np.ascontiguousarray(big_e[:, :n]), mode=EF)
    assert np.array_equal(lm, lm_c) and np.array_equal(cnt, cnt_c)
    w = np.zeros(n, np.float32)
    oracle.step(w, big_g[:, :n], big_e[:, :n], 0.1, mode=EF)
    assert np.isnan(big_g[:, n:]).all() and np.isnan(big_e[:, n:]).all()   # padding untouched
    assert np.isfinite(big_e[:, :n]).all() and np.isfinite(w).all()


def test_subnormal_negative_stays_negative():
    tiny = np.float32(-1e-45)  # smallest-magnitude negative subnormal
    v = np.array([[tiny, 1.0, 2.0]], np.float32)
    lm, cnt, mask = oracle.encode(v, None, mode=ALG1, want_mask=True)
    assert cnt.tolist() == [2] and mask.tolist() == [[6]]
    assert lm[0, 1] == np.float32(1e-45)


def test_rejects_bad_arguments():
    g = np.zeros((1, 4), np.float32)
    with pytest.raises(RuntimeError):
        oracle.encode(g, None, mode=EF)            # EF needs the error buffer
    with pytest.raises(ValueError):
        oracle.encode(g.astype(np.float64), None, mode=ALG1)


# ---------------------------------------------------------------- Algorithm 1 lines 9-10 (dense step)
def test_dense_sync_matches_numpy_mean_axpy_and_special_cases():
    rng = np.random.default_rng(31)
    P, n, lr = 5, 20011, 0.3
    g = (rng.standard_normal((P, n)) * 1e-2).astype(np.float32)
    w0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    ref = w0.astype(np.float64) - np.float64(np.float32(lr)) * g.astype(np.float64).mean(axis=0)
    w = w0.copy()
    oracle.dense_sync(w, g, lr)
    assert np.max(np.abs(w - ref)) <= 1.01 * np.spacing(np.abs(w0).max())
    # every replica receives the same averaged update (this is what re-synchronises the workers)
    w_rep = np.tile(w0, (P, 1)) + np.arange(P, dtype=np.float32)[:, None]
    oracle.dense_sync(w_rep, g, lr)
    for p in range(P):
        assert np.max(np.abs(w_rep[p] - (ref + p))) <= 1.01 * np.spacing(np.float32(p + 1))
    # P = 1 is plain SGD; identical workers give the single-worker result
    w1 = w0.copy()
    oracle.dense_sync(w1, g[:1], lr)
    ref1 = w0.astype(np.float64) - np.float64(np.float32(lr)) * g[0].astype(np.float64)
    assert np.max(np.abs(w1 - ref1)) <= 1.01 * np.spacing(np.abs(w0).max())
    w2 = w0.copy()
    oracle.dense_sync(w2, np.tile(g[:1], (4, 1)), lr)
    assert np.array_equal(w2, w1)


@pytest.mark.parametrize("seed", range(10))
def test_dense_sync_bruteforce_rational(seed):
    rng = np.random.default_rng(seed)
    n, P = int(rng.integers(1, 9)), int(rng.integers(1, 6))
    g = rng.standard_normal((P, n)).astype(np.float32)
    w0 = rng.standard_normal(n).astype(np.float32)
    w = w0.copy()
    oracle.dense_sync(w, g, 0.125)
    for i in range(n):
        mean = sum((Fraction(float(g[p, i])) for p in range(P)), Fraction(0)) / P
        assert _ulp_close(w[i], _round32(Fraction(float(w0[i])) - Fraction(1, 8) * mean))


def test_dense_sync_after_identical_local_steps_equals_eq1():
    """Eq. 1: one dense step from a common w is w - lr * (1/P) sum_p g^p; with hand numbers."""
    g = _f32([[1, -2, 4], [3, 2, -8]])
    w = np.array([10, 10, 10], np.float32)
    oracle.dense_sync(w, g, 0.5)
    assert w.tolist() == [9.0, 10.0, 11.0]


# ---------------------------------------------------------------- momentum / weight decay on the reconstructed gradient
def test_golden_m1_momentum_and_weight_decay_two_steps():
    fx = _load("m1_momentum_weight_decay_two_steps.json")
    for case in fx["cases"]:
        w = np.array(fx["w0"], np.float32)
        m = np.array(fx["m0"], np.float32)
        e = _f32(fx["e0"])
        for t in range(2):
            g = _f32(fx["g"][t])
            oracle.step_momentum(w, m, g, e, fx["lr"], case["beta"], case["weight_decay"], mode=EF)
            assert e.tolist() == fx["e"][t]
            assert m.tolist() == case["m"][t]
            assert w.tolist() == case["w"][t]


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
def test_momentum_with_beta_zero_and_no_decay_is_the_plain_step_bit_for_bit(mode, replicated):
    rng = np.random.default_rng(11)
    P, n = 3, 257
    g = (rng.standard_normal((P, n)) * 1e-2).astype(np.float32)
    e0 = (rng.standard_normal((P, n)) * 3e-3).astype(np.float32)
    w0 = (rng.standard_normal((P, n) if replicated else n) * 0.02).astype(np.float32)
    lm, cnt, _ = oracle.encode(g, e0 if mode == EF else None, mode=mode)
    gm = oracle.global_average(lm)
    w_a, e_a = w0.copy(), e0.copy()
    oracle.decode_update(w_a, g, e_a, lm, gm, 0.1, mode=mode)
    w_b, e_b = w0.copy(), e0.copy()
    m = (rng.standard_normal(w0.shape)).astype(np.float32)       # beta = 0: the old buffer must not matter
    oracle.decode_update_momentum(w_b, m, g, e_b, lm, gm, 0.1, 0.0, 0.0, mode=mode)
    assert np.array_equal(w_a, w_b) and np.array_equal(e_a, e_b)
    # and the buffer now holds g_hat itself: w0 - lr*m reproduces w up to the two roundings
    assert np.allclose(w0.astype(np.float64) - np.float32(0.1).astype(np.float64) * m, w_b, rtol=0, atol=1e-8)


def test_momentum_constant_gradient_closed_form():
    """A two-valued gradient with e = 0 and one worker is reconstructed exactly (g_hat = g, no
    residual), so every step feeds the same g_hat: m_t = g_hat (1 - beta^t) / (1 - beta) and
    w_t = w_0 - lr * sum_{s<=t} m_s."""
    n, beta, lr, T = 64, 0.5, 0.25, 6
    g = np.where(np.arange(n) % 3 == 0, 0.75, -0.5).astype(np.float32)[None, :]
    w = np.linspace(-1, 1, n).astype(np.float32)
    w0 = w.astype(np.float64).copy()
    m = np.zeros(n, np.float32)
    e = np.zeros((1, n), np.float32)
    acc = np.zeros(n)
    for t in range(1, T + 1):
        oracle.step_momentum(w, m, g, e, lr, beta, 0.0, mode=EF)
        assert not e.any()
        m_exact = g[0].astype(np.float64) * (1 - beta ** t) / (1 - beta)
        acc += m_exact
        assert np.allclose(m, m_exact, rtol=1e-7, atol=0)
        assert np.allclose(w, w0 - lr * acc, rtol=0, atol=2e-7)


def test_weight_decay_alone_shrinks_the_weights():
    """beta = 0: w <- w (1 - lr*wd) - lr*g_hat."""
    rng = np.random.default_rng(5)
    P, n, lr, wd = 2, 100, 0.5, 0.125
    g = rng.standard_normal((P, n)).astype(np.float32)
    e = np.zeros((P, n), np.float32)
    w0 = rng.standard_normal(n).astype(np.float32)
    w_plain, e1 = w0.copy(), e.copy()
    oracle.step(w_plain, g, e1, lr, mode=EF)
    ghat_mean = (w0.astype(np.float64) - w_plain) / lr
    w, m, e2 = w0.copy(), np.zeros(n, np.float32), e.copy()
    oracle.step_momentum(w, m, g, e2, lr, 0.0, wd, mode=EF)
    assert np.allclose(w, w0.astype(np.float64) * (1 - lr * wd) - lr * ghat_mean, rtol=0, atol=1e-6)
    assert np.array_equal(e1, e2)


@pytest.mark.parametrize("seed", range(12))
def test_momentum_bruteforce_rational(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 17))
    P = int(rng.integers(1, 5))
    mode = EF if seed % 2 == 0 else ALG1
    g = (rng.standard_normal((P, n)) * 10.0 ** rng.uniform(-3, 1)).astype(np.float32)
    e = (rng.standard_normal((P, n)) * 10.0 ** rng.uniform(-3, 1)).astype(np.float32)
    lr, beta, wd = np.float32(0.3), np.float32(0.9), np.float32(5e-4)
    v = (g + e).astype(np.float32) if mode == EF else g
    lm, _, _ = oracle.encode(g, e if mode == EF else None, mode=mode)
    gm = oracle.global_average(lm)
    F = lambda x: Fraction(float(x))
    ghat = [[None] * n for _ in range(P)]
    for p in range(P):
        for i in range(n):
            mean_vec = F(gm[0]) if v[p, i] >= 0 else -F(gm[1])
            if mode == EF:
                ghat[p][i] = mean_vec
            else:
                enc = F(lm[p, 0]) if v[p, i] >= 0 else -F(lm[p, 1])
                ghat[p][i] = F(v[p, i]) - enc + mean_vec
    w0 = rng.standard_normal(n).astype(np.float32)
    m0 = rng.standard_normal(n).astype(np.float32)
    # one shared w: the worker-mean of g_hat drives one momentum vector
    w, m, e_sh = w0.copy(), m0.copy(), e.copy()
    oracle.decode_update_momentum(w, m, g, e_sh, lm, gm, lr, beta, wd, mode=mode)
    for i in range(n):
        u = sum((ghat[p][i] for p in range(P)), Fraction(0)) / P + F(wd) * F(w0[i])
        m_new = F(beta) * F(m0[i]) + u
        assert _ulp_close(m[i], _round32(m_new))
        assert _ulp_close(w[i], _round32(F(w0[i]) - F(lr) * m_new))
    # one replica per worker: its own g_hat, its own momentum vector
    w_r, m_r, e_r = np.tile(w0, (P, 1)), np.tile(m0, (P, 1)), e.copy()
    oracle.decode_update_momentum(w_r, m_r, g, e_r, lm, gm, lr, beta, wd, mode=mode)
    for p in range(P):
        for i in range(n):
            m_new = F(beta) * F(m0[i]) + ghat[p][i] + F(wd) * F(w0[i])
            assert _ulp_close(m_r[p, i], _round32(m_new))
            assert _ulp_close(w_r[p, i], _round32(F(w0[i]) - F(lr) * m_new))
    assert np.array_equal(e_sh, e_r)
    # the shared state is the mean of the replica states (the update is linear)
    assert np.allclose(w, w_r.astype(np.float64).mean(0), rtol=0, atol=1e-6 * max(1.0, float(np.abs(w0).max())))
    assert np.allclose(m, m_r.astype(np.float64).mean(0), rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------- the OpenMP timing copy of the step
@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("shared", [True, False])
def test_all_cores_copy_agrees_with_the_pinned_oracle(mode, shared):
    """bench.py times an OpenMP copy of the step next to the single-threaded oracle; the copy is
    held to the pinned oracle here (it may differ only in the order of the fp64 additions)."""
    rng = np.random.default_rng(17)
    P, n = 3, 200_003
    g = (rng.standard_normal((P, n)) * 1e-3).astype(np.float32)
    g[rng.random((P, n)) < 0.05] = 0.0
    e = (rng.standard_normal((P, n)) * 3e-4).astype(np.float32)
    w = (rng.standard_normal(n if shared else (P, n)) * 0.02).astype(np.float32)
    w1, e1 = w.copy(), e.copy()
    lm1, gm1, c1 = oracle.step(w1, g, e1, 0.1, mode=mode)
    w2, e2 = w.copy(), e.copy()
    lm2, gm2, c2 = oracle.step_all_cores(w2, g, e2, 0.1, mode=mode)
    assert np.array_equal(c1, c2)
    assert np.allclose(lm1, lm2, rtol=2e-7, atol=0) and np.allclose(gm1, gm2, rtol=2e-7, atol=0)
    assert np.allclose(w1, w2, rtol=0, atol=1e-9) and np.allclose(e1, e2, rtol=0, atol=1e-9)
    assert oracle.omp_threads() >= 1
