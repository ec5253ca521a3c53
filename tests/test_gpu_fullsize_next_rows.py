"""The rows beyond the plain step at full benchmark sizes, every element compared with the oracle:
the momentum / weight-decay step (c4), the segment-list step and its per-tensor variant (c3, 161
tensors at full length), the dense synchronisation step (c4), bfloat16 gradients (c2) and the
general-alignment kernels (c4 with row stride n + 1)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from paper_2006_07405_b200 import workloads as W
from parity_util import (STATE_TOL, assert_means, device_outliers, oracle_decode_by_chunks, oracle_encode_by_worker,
                         tau_err, tau_w)

pytestmark = pytest.mark.gpu
EF = B.MODE_EF


def _all_elements(what, got_w, w_ref, got_e, e_ref, gm_ref, allowed=0):
    bad, worst = device_outliers(got_w, w_ref, tau_w(w_ref))
    assert bad <= allowed, f"{what} w: {bad} elements over {STATE_TOL} (worst {worst:.3e})"
    for p in range(e_ref.shape[0]):
        bad, worst = device_outliers(got_e[p], e_ref[p], tau_err(gm_ref))
        assert bad <= allowed, f"{what} err of worker {p}: {bad} elements over {STATE_TOL} (worst {worst:.3e})"


def test_momentum_step_c4_full_size_two_steps():
    wl = W.get_workload("c4_vgg16")
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, "cuda")
    e = B.padded_rows(P, n, "cuda", fill=0.0)
    w = torch.empty(n, device="cuda")
    m = torch.zeros(n, device="cuda")
    W.init_weights(wl, w)
    w_ref, m_ref, e_ref = w.cpu().numpy(), np.zeros(n, np.float32), np.zeros((P, n), np.float32)
    ctx = B.a2sgd_create(n, P, 0, EF)
    beta, wd = 0.9, 1e-4
    for step in range(2):
        W.fill_gradients(wl, step, g)
        g_np = g.cpu().numpy()
        B.a2sgd_step_momentum(ctx, w, m, g, e, wl.lr, beta, wd)
        lm_ref, cnt_ref, _ = oracle_encode_by_worker(oracle, g_np, e_ref, oracle.MODE_EF)
        gm_ref = oracle.global_average(lm_ref)
        oracle_decode_by_chunks(oracle, w_ref, g_np, e_ref, lm_ref, gm_ref, wl.lr, oracle.MODE_EF,
                                mom=m_ref, beta=beta, wd=wd)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        if step == 0:
            assert np.array_equal(cnt, cnt_ref)
        assert_means(lm, lm_ref)
        assert_means(gm, gm_ref)
        allowed = 0 if step == 0 else max(2, n * P // 1_000_000)
        _all_elements(f"momentum step {step}", w, w_ref, e, e_ref, gm_ref, allowed)
        bad, worst = device_outliers(m, m_ref, tau_err(gm_ref) / (1 - beta))
        assert bad <= allowed, f"momentum buffer step {step}: {bad} elements off (worst {worst:.3e})"
    ctx.destroy()


@pytest.mark.parametrize("per_tensor", [False, True])
def test_segment_list_c3_full_size(per_tensor):
    """161 tensors at their full lengths (64 ... 2,359,296 elements), P = 8, every element."""
    wl = W.get_workload("c3_resnet50")
    n, P = wl.n, wl.P
    sizes = [s.numel for s in wl.segments]
    flat_g = B.padded_rows(P, n, "cuda")
    W.fill_gradients(wl, 0, flat_g)
    gen = torch.Generator("cuda").manual_seed(5)
    flat_e = B.padded_rows(P, n, "cuda").normal_(0.0, 1e-4, generator=gen)
    flat_w = torch.empty(n, device="cuda")
    W.init_weights(wl, flat_w)
    grad = [[t.clone() for t in torch.split(flat_g[p], sizes)] for p in range(P)]
    err = [[t.clone() for t in torch.split(flat_e[p], sizes)] for p in range(P)]
    w = [t.clone() for t in torch.split(flat_w, sizes)]
    g_np, e_ref, w_ref = flat_g.cpu().numpy(), flat_e.cpu().numpy(), flat_w.cpu().numpy()
    ctx = B.a2sgd_create(n, P, 0, EF)
    plan = B.a2sgd_segments_create(ctx, grad, err, w)
    if per_tensor:
        B.a2sgd_step_segments_per_tensor(ctx, plan, wl.lr)
        lm_all, gm_all, cnt_all = B.a2sgd_read_segment_stats(ctx, plan, len(sizes))
        off = 0
        for k, s in enumerate(sizes):                       # reference: one oracle step per tensor
            g_k = np.ascontiguousarray(g_np[:, off:off + s])
            e_k = np.ascontiguousarray(e_ref[:, off:off + s])
            w_k = w_ref[off:off + s].copy()
            lm, gm, cnt = oracle.step(w_k, g_k, e_k, wl.lr, mode=oracle.MODE_EF)
            assert np.array_equal(cnt_all[k], cnt)
            assert_means(lm_all[k], lm, f"tensor {k}")
            assert_means(gm_all[k], gm, f"tensor {k}")
            bad, worst = device_outliers(w[k], w_k, tau_w(w_ref))
            assert bad == 0, f"tensor {k} w: {bad} off (worst {worst:.3e})"
            for p in range(P):
                bad, worst = device_outliers(err[p][k], e_k[p], tau_err(gm))
                assert bad == 0, f"tensor {k} err of worker {p}: {bad} off (worst {worst:.3e})"
            off += s
    else:
        B.a2sgd_step_segments(ctx, plan, wl.lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        lm_ref, cnt_ref, _ = oracle_encode_by_worker(oracle, g_np, e_ref, oracle.MODE_EF)
        gm_ref = oracle.global_average(lm_ref)
        oracle_decode_by_chunks(oracle, w_ref, g_np, e_ref, lm_ref, gm_ref, wl.lr, oracle.MODE_EF)
        assert status == B.OK and np.array_equal(cnt, cnt_ref)
        assert_means(lm, lm_ref)
        assert_means(gm, gm_ref)
        _all_elements("segments", torch.cat(w), w_ref, [torch.cat(err[p]) for p in range(P)], e_ref, gm_ref)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    plan.destroy()
    ctx.destroy()


def test_dense_sync_c4_full_size():
    wl = W.get_workload("c4_vgg16")
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, "cuda")
    W.fill_gradients(wl, 2, g)
    w = torch.empty(n, device="cuda")
    W.init_weights(wl, w)
    w_ref = w.cpu().numpy()
    g_np = g.cpu().numpy()
    ctx = B.a2sgd_create(n, P, 0, EF)
    B.a2sgd_dense_sync(ctx, w, g, wl.lr)
    oracle.dense_sync(w_ref, g_np, wl.lr)
    bad, worst = device_outliers(w, w_ref, tau_w(w_ref))
    assert bad == 0, f"{bad} elements off (worst {worst:.3e})"
    ctx.destroy()


def test_bf16_gradients_c2_full_size():
    wl = W.get_workload("c2_lstm_ptb")
    n, P = wl.n, wl.P
    g32 = B.padded_rows(P, n, "cuda")
    W.fill_gradients(wl, 0, g32)
    g16 = torch.empty((P, g32.stride(0)), dtype=torch.bfloat16, device="cuda")[:, :n]
    g16.copy_(g32)
    e = B.padded_rows(P, n, "cuda", fill=0.0)
    w = torch.empty(n, device="cuda")
    W.init_weights(wl, w)
    g_np = g16.float().cpu().numpy()                       # widening is exact
    e_ref, w_ref = np.zeros((P, n), np.float32), w.cpu().numpy()
    ctx = B.a2sgd_create(n, P, 0, EF)
    B.a2sgd_step_bf16(ctx, w, g16, e, wl.lr)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, cnt_ref, _ = oracle_encode_by_worker(oracle, g_np, e_ref, oracle.MODE_EF)
    gm_ref = oracle.global_average(lm_ref)
    oracle_decode_by_chunks(oracle, w_ref, g_np, e_ref, lm_ref, gm_ref, wl.lr, oracle.MODE_EF)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    _all_elements("bf16", w, w_ref, e, e_ref, gm_ref)
    ctx.destroy()


def test_misaligned_rows_c4_full_size():
    """Row stride n + 1: every row at a different 4-byte phase (the general-alignment kernels)."""
    wl = W.get_workload("c4_vgg16")
    n, P = wl.n, wl.P
    g = torch.empty((P, n + 1), device="cuda")[:, :n]
    e = torch.zeros((P, n + 1), device="cuda")[:, :n]
    W.fill_gradients(wl, 1, g)
    w = torch.empty(n + 3, device="cuda")[3:]
    W.init_weights(wl, w)
    g_np, e_ref, w_ref = g.cpu().numpy(), np.zeros((P, n), np.float32), w.cpu().numpy()
    ctx = B.a2sgd_create(n, P, 0, EF)
    B.a2sgd_step(ctx, w, g, e, wl.lr)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, cnt_ref, _ = oracle_encode_by_worker(oracle, g_np, e_ref, oracle.MODE_EF)
    gm_ref = oracle.global_average(lm_ref)
    oracle_decode_by_chunks(oracle, w_ref, g_np, e_ref, lm_ref, gm_ref, wl.lr, oracle.MODE_EF)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    _all_elements("misaligned", w, w_ref, [e[p].contiguous() for p in range(P)], e_ref, gm_ref)
    ctx.destroy()
