"""The host-thread helpers of the full-size GPU comparisons return exactly what single oracle calls
return (they only split the calls: per worker for the encode, per element range for the decode)."""
import numpy as np
import pytest

import oracle
from parity_util import oracle_decode_by_chunks, oracle_encode_by_worker, strict_rel_err


@pytest.mark.parametrize("mode", [oracle.MODE_EF, oracle.MODE_ALG1])
@pytest.mark.parametrize("shared", [True, False])
def test_split_calls_equal_single_calls(mode, shared):
    rng = np.random.default_rng(3)
    P, n = 3, 100_003
    g = (rng.standard_normal((P, n)) * 1e-3).astype(np.float32)
    e = (rng.standard_normal((P, n)) * 1e-4).astype(np.float32)
    w = (rng.standard_normal(n if shared else (P, n)) * 0.02).astype(np.float32)
    err = e if mode == oracle.MODE_EF else None
    lm, cnt, mask = oracle.encode(g, err, mode=mode, want_mask=True)
    lm2, cnt2, mask2 = oracle_encode_by_worker(oracle, g, err, mode, want_mask=True)
    assert np.array_equal(lm, lm2) and np.array_equal(cnt, cnt2) and np.array_equal(mask, mask2)
    gm = oracle.global_average(lm)
    w1, e1 = w.copy(), e.copy()
    oracle.decode_update(w1, g, e1, lm, gm, 0.1, mode=mode)
    w2, e2 = w.copy(), e.copy()
    oracle_decode_by_chunks(oracle, w2, g, e2, lm, gm, 0.1, mode, chunks=7)
    assert np.array_equal(w1, w2) and np.array_equal(e1, e2)
    m1, m2 = np.zeros_like(w), np.zeros_like(w)
    w3, e3 = w.copy(), e.copy()
    oracle.decode_update_momentum(w3, m1, g, e3, lm, gm, 0.1, 0.9, 1e-3, mode=mode)
    w4, e4 = w.copy(), e.copy()
    oracle_decode_by_chunks(oracle, w4, g, e4, lm, gm, 0.1, mode, chunks=5, mom=m2, beta=0.9, wd=1e-3)
    assert np.array_equal(w3, w4) and np.array_equal(m1, m2) and np.array_equal(e3, e4)


def test_strict_relative_error_skips_zero_references():
    assert strict_rel_err([1.0, 2.0, 5.0], [1.0, 0.0, 4.0]) == 0.25
