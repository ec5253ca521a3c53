"""GPU parity of the momentum / weight-decay form of the update (a2sgd_step_momentum,
a2sgd_decode_update_momentum) against the oracle's decode_update_momentum, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from paper_2006_07405_b200 import workloads as W
from parity_util import STATE_TOL, assert_means, assert_state, normalised_err, tau_err

pytestmark = pytest.mark.gpu

EF, ALG1 = B.MODE_EF, B.MODE_ALG1


def _rows(P, n, stride, off, device="cuda"):
    """[P, n] view with the given row stride whose first element sits ``off`` floats past a
    256-byte boundary (torch allocations are at least 256-byte aligned)."""
    buf = torch.zeros(off + P * stride + 8, device=device)
    return buf[off: off + P * stride].view(P, stride)[:, :n], buf


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("n,P,pad,off", [(1, 1, 0, 0), (37, 3, 0, 0), (1025, 2, 7, 0), (4099, 4, 5, 0),
                                         (65536 + 7, 8, 1, 0), (70001, 4, 3, 4), (70001, 5, 0, 1),
                                         ((1 << 20) + 1, 4, 31, 0)])
def test_momentum_steps_match_oracle(mode, replicated, n, P, pad, off):
    stride = n + pad
    rng = np.random.default_rng(n * 31 + P)
    g_dev, _ = _rows(P, n, stride, off)
    e_dev, _ = _rows(P, n, stride, off)
    w_dev, w_raw = _rows(P if replicated else 1, n, stride, off)
    m_dev, m_raw = _rows(P if replicated else 1, n, stride, off)
    w0 = (rng.standard_normal((P if replicated else 1, n)) * 0.02).astype(np.float32)
    w_dev.copy_(torch.from_numpy(w0))
    if not replicated:
        w_dev, m_dev = w_dev[0], m_dev[0]
    w_ref = w0.copy() if replicated else w0[0].copy()
    m_ref = np.zeros_like(w_ref)
    e_ref = np.zeros((P, n), np.float32)
    lr, beta, wd = 0.1, 0.9, 5e-4
    ctx = B.a2sgd_create(n, P, 0, mode)
    for step in range(3):
        g = (rng.standard_normal((P, n)) * 1e-3).astype(np.float32)
        g_dev.copy_(torch.from_numpy(g))
        err_arg = e_dev if (mode == EF or step % 2 == 0) else None      # ALG1: eps is optional
        B.a2sgd_step_momentum(ctx, w_dev, m_dev, g_dev, err_arg, lr, beta, wd)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        lm_ref, gm_ref, cnt_ref = oracle.step_momentum(w_ref, m_ref, g, e_ref, lr, beta, wd, mode=mode)
        if step == 0 or mode == ALG1:
            assert np.array_equal(cnt, cnt_ref)
        assert_means(lm, lm_ref)
        assert_means(gm, gm_ref)
        flips = max(2, n * P // 10 ** 6) if (step > 0 and mode == EF) else 0
        e_got = e_dev.cpu().numpy() if err_arg is not None else None
        assert_state(w_dev.cpu().numpy(), w_ref, e_got, e_ref, gm_ref, f"step {step}", max_outliers=flips)
        tau_m = tau_err(gm_ref) / (1.0 - beta)
        bad = int(np.count_nonzero(np.abs(m_dev.cpu().numpy().astype(np.float64) - m_ref)
                                   > STATE_TOL * np.maximum(np.abs(m_ref), tau_m)))
        assert bad <= flips, f"momentum buffer: {bad} elements off"
    # nothing outside the live elements of w / mom was written
    for raw, rows in ((w_raw, P if replicated else 1), (m_raw, P if replicated else 1)):
        buf = raw.cpu().numpy()
        live = np.zeros(buf.shape, bool)
        for r in range(rows):
            live[off + r * stride: off + r * stride + n] = True
        assert not buf[~live].any()
    ctx.destroy()


@pytest.mark.parametrize("replicated", [False, True])
def test_zero_coefficients_give_the_plain_step_bit_for_bit(replicated):
    n, P = 300_007, 4
    gen = torch.Generator("cuda").manual_seed(3)
    g = B.padded_rows(P, n, "cuda").normal_(0, 1e-3, generator=gen)
    e0 = B.padded_rows(P, n, "cuda").normal_(0, 3e-4, generator=gen)
    w0 = (B.padded_rows(P, n, "cuda") if replicated else torch.empty(n, device="cuda")).normal_(0, 0.02, generator=gen)
    ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_TWO_PASS)
    w_a, e_a = w0.clone(), e0.clone()
    B.a2sgd_step(ctx, w_a, g, e_a, 0.1)
    w_b, e_b = w0.clone(), e0.clone()
    m = torch.ones_like(w0)                      # beta = 0: the old buffer must not matter
    B.a2sgd_step_momentum(ctx, w_b, m, g, e_b, 0.1, 0.0, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(e_a, e_b)
    # w differs from the plain step only by the rounding of lr * g_hat done in two steps instead of one fma
    assert normalised_err(w_b.cpu().numpy(), w_a.cpu().numpy(), float(w0.abs().mean())) <= 1e-6
    ctx.destroy()


def test_staged_call_and_bad_arguments():
    n, P = 4096, 2
    g = torch.randn(P, n, device="cuda") * 1e-3
    e = torch.zeros(P, n, device="cuda")
    w = torch.randn(n, device="cuda") * 0.02
    m = torch.zeros(n, device="cuda")
    ctx = B.a2sgd_create(n, P, 0, EF)
    lm = torch.zeros(P, 2, device="cuda")
    gm = torch.zeros(2, device="cuda")
    g_h, e_h, w_h, m_h = g.cpu().numpy(), e.cpu().numpy(), w.cpu().numpy(), m.cpu().numpy()
    B.a2sgd_encode(ctx, g, e, lm)
    B.a2sgd_global_average(ctx, lm, gm)
    B.a2sgd_decode_update_momentum(ctx, w, m, g, e, lm, gm, 0.1, 0.5, 0.01)
    lm_ref, gm_ref, _ = oracle.step_momentum(w_h, m_h, g_h, e_h, 0.1, 0.5, 0.01, mode=oracle.MODE_EF)
    assert_state(w.cpu().numpy(), w_h, e.cpu().numpy(), e_h, gm_ref, "staged")
    assert normalised_err(m.cpu().numpy(), m_h, tau_err(gm_ref)) <= STATE_TOL
    for kwargs, status in (({"beta": 1.0}, B.ERR_ARG), ({"beta": -0.1}, B.ERR_ARG), ({"wd": -1.0}, B.ERR_ARG),
                           ({"beta": float("nan")}, B.ERR_ARG)):
        with pytest.raises(B.A2SGDError) as ei:
            B.a2sgd_step_momentum(ctx, w, m, g, e, 0.1, kwargs.get("beta", 0.9), kwargs.get("wd", 0.0))
        assert ei.value.status == status
    with pytest.raises(B.A2SGDError) as ei:       # momentum buffer must have the layout of w
        B.a2sgd_step_momentum(ctx, w, torch.zeros(P, n, device="cuda"), g, e, 0.1, 0.9, 0.0)
    assert ei.value.status == B.ERR_ARG
    ctx.destroy()


def test_momentum_c2_div4_five_steps_free_running():
    """A case spanning many CTAs in the launch configuration the bench times (aligned rows, P = 4)."""
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 4)
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, "cuda")
    e = B.padded_rows(P, n, "cuda", fill=0.0)
    w = torch.empty(n, device="cuda")
    m = torch.zeros(n, device="cuda")
    W.init_weights(wl, w)
    w_ref, m_ref, e_ref = w.cpu().numpy(), np.zeros(n, np.float32), np.zeros((P, n), np.float32)
    ctx = B.a2sgd_create(n, P, 0, EF)
    for step in range(5):
        W.fill_gradients(wl, step, g)
        g_h = g.cpu().numpy()
        B.a2sgd_step_momentum(ctx, w, m, g, e, wl.lr, 0.9, 1e-4)
        lm_ref, gm_ref, _ = oracle.step_momentum(w_ref, m_ref, g_h, e_ref, wl.lr, 0.9, 1e-4, mode=oracle.MODE_EF)
        lm, gm, _, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        assert_means(lm, lm_ref)
        assert_means(gm, gm_ref)
        flips = max(2, n * P // 10 ** 6) if step else 0
        assert_state(w.cpu().numpy(), w_ref, e.cpu().numpy(), e_ref, gm_ref, f"step {step}", max_outliers=flips)
    ctx.destroy()
