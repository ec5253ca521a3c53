"""The opt-in deferred-residual representation: the error buffer holds v between steps and the
residual is formed one step late.  Same fp32 operations as the default path, so weights and (after
materialising) residuals must be BIT-identical to it, and within tolerance of the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from paper_2006_07405_b200 import workloads as W
from parity_util import assert_means, assert_state

pytestmark = pytest.mark.gpu
EF = B.MODE_EF


def _rows(P, n, gen, scale):
    t = B.padded_rows(P, n, "cuda")
    t.normal_(0.0, scale, generator=gen)
    return t


@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,n", [(1, 5), (1, 100_003), (3, 31), (4, 32), (4, 250_016), (4, 333_333), (8, 70_001), (5, 4097)])
def test_deferred_is_bit_identical_to_default_and_matches_oracle(replicated, P, n):
    gen = torch.Generator("cuda").manual_seed(P * 1000 + n)
    steps = 4
    grads = [_rows(P, n, gen, 1e-3) for _ in range(steps)]
    e0 = _rows(P, n, gen, 2e-4)
    w0 = _rows(P, n, gen, 0.02) if replicated else torch.randn(n, device="cuda", generator=gen) * 0.02

    def clone_w():
        if replicated:
            w = B.padded_rows(P, n, "cuda"); w.copy_(w0); return w
        return w0.clone()

    def clone_e():
        e = B.padded_rows(P, n, "cuda"); e.copy_(e0); return e

    ref_ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_TWO_PASS)
    dfr_ctx = B.a2sgd_create(n, P, 0, EF | B.DEFERRED_RESIDUAL)
    w_ref, e_ref, w_d, e_d = clone_w(), clone_e(), clone_w(), clone_e()
    wh, eh = w0.cpu().numpy().copy(), e0.cpu().numpy().copy()
    for k in range(steps):
        B.a2sgd_step(ref_ctx, w_ref, grads[k], e_ref, 0.1)
        B.a2sgd_step(dfr_ctx, w_d, grads[k], e_d, 0.1)
        r = B.a2sgd_read_stats(ref_ctx)
        d = B.a2sgd_read_stats(dfr_ctx)
        assert d[3] == B.OK
        assert np.array_equal(r[0], d[0]) and np.array_equal(r[1], d[1]) and np.array_equal(r[2], d[2])
        assert torch.equal(w_ref, w_d), f"w differs at step {k}"
        lm_o, gm_o, cnt_o = oracle.step(wh, grads[k].cpu().numpy(), eh, 0.1, mode=oracle.MODE_EF)
        if k == 0:
            assert np.array_equal(d[2], cnt_o)
        assert_means(d[0], lm_o)
        assert_means(d[1], gm_o)
        if k == 1:   # leave and re-enter the deferred form in the middle of the run
            B.a2sgd_materialize_err(dfr_ctx, e_d)
            assert torch.equal(e_ref, e_d), "materialised residual differs"
    B.a2sgd_materialize_err(dfr_ctx, e_d)
    B.a2sgd_materialize_err(dfr_ctx, e_d)          # second call is a no-op
    torch.cuda.synchronize()
    assert torch.equal(e_ref, e_d)
    assert_state(w_d.cpu().numpy(), wh, e_d.cpu().numpy(), eh, gm_o, f"deferred P={P} n={n}", max_outliers=2)
    ref_ctx.destroy()
    dfr_ctx.destroy()


def test_deferred_mode_argument_rules():
    n, P = 1000, 2
    with pytest.raises(B.A2SGDError):
        B.a2sgd_create(n, P, 0, B.MODE_ALG1 | B.DEFERRED_RESIDUAL)       # error feedback only
    ctx = B.a2sgd_create(n, P, 0, EF | B.DEFERRED_RESIDUAL)
    g = torch.zeros((P, n + 1), device="cuda")[:, :n]                       # row stride not a multiple of 8
    e = torch.zeros((P, n + 1), device="cuda")[:, :n]
    w = torch.zeros(n, device="cuda")
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_step(ctx, w, g, e, 0.1)
    assert ei.value.status == B.ERR_ALIGN
    lm = torch.zeros((P, 2), device="cuda")
    g2, e2 = B.padded_rows(P, n, "cuda", 0.0), B.padded_rows(P, n, "cuda", 0.0)
    with pytest.raises(B.A2SGDError) as ei:                                 # staged calls assume a true residual
        B.a2sgd_encode(ctx, g2, e2, lm)
    assert ei.value.status == B.ERR_ARG
    ctx.destroy()


def test_deferred_full_size_c2_against_default():
    wl = W.get_workload("c2_lstm_ptb")
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, "cuda")
    outs = []
    for flags in (EF | B.FORCE_TWO_PASS, EF | B.DEFERRED_RESIDUAL):
        e = B.padded_rows(P, n, "cuda", fill=0.0)
        w = torch.empty(n, device="cuda")
        W.init_weights(wl, w)
        ctx = B.a2sgd_create(n, P, 0, flags)
        for step in range(3):
            W.fill_gradients(wl, step, g)
            B.a2sgd_step(ctx, w, g, e, wl.lr)
        if flags & B.DEFERRED_RESIDUAL:
            B.a2sgd_materialize_err(ctx, e)
        stats = B.a2sgd_read_stats(ctx)
        outs.append((w, e, stats))
        ctx.destroy()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert np.array_equal(outs[0][2][0], outs[1][2][0]) and np.array_equal(outs[0][2][2], outs[1][2][2])
