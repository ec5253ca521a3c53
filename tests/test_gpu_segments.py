"""Segment-list entry points: the model as separate tensors (any alignment), reduced to the same
whole-model means as the flat path.  Reference: the CPU oracle on the concatenation."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from paper_2006_07405_b200 import workloads as W
from parity_util import assert_means, assert_state

pytestmark = pytest.mark.gpu
EF, ALG1 = B.MODE_EF, B.MODE_ALG1


def _tensors(sizes, offsets, gen, scale):
    """One tensor per size; tensor k starts offsets[k % len(offsets)] elements into its own allocation."""
    out = []
    for k, n in enumerate(sizes):
        o = offsets[k % len(offsets)]
        buf = torch.full((n + o + 8,), float("nan"), device="cuda")
        t = buf[o:o + n]
        t.normal_(0.0, scale, generator=gen)
        out.append(t)
    return out


def _cat(rows):
    return np.stack([torch.cat(r).cpu().numpy() for r in rows])


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,offsets", [(1, [0]), (4, [0]), (3, [0, 1, 0, 8, 3]), (8, [0, 0, 0, 2]), (2, [1])])
def test_segment_list_step_matches_oracle_on_concatenation(mode, replicated, P, offsets):
    wl = W.scaled(W.get_workload("c3_resnet50"), 16)        # 161 tensors, many of them tiny
    sizes = [s.numel for s in wl.segments] + [1, 2, 7, 2047, 2048, 2049, 4096 + 8]
    n = sum(sizes)
    gen = torch.Generator("cuda").manual_seed(P * 100 + len(offsets))
    grad = [_tensors(sizes, offsets, gen, 1e-3) for _ in range(P)]
    err = [_tensors(sizes, offsets, gen, 3e-4) for _ in range(P)]
    w = [_tensors(sizes, offsets, gen, 0.02) for _ in range(P if replicated else 1)]
    gh, eh = _cat(grad), _cat(err)
    wh = _cat(w) if replicated else _cat(w)[0]
    ctx = B.a2sgd_create(n, P, 0, mode)
    plan = B.a2sgd_segments_create(ctx, grad, err, w if replicated else w[0], w_replicated=replicated)
    B.a2sgd_step_segments(ctx, plan, 0.1)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, gm_ref, cnt_ref = oracle.step(wh, gh, eh, 0.1, mode=mode)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    w_got = _cat(w) if replicated else _cat(w)[0]
    assert_state(w_got, wh, _cat(err), eh, gm_ref, f"segments P={P}")
    assert np.array_equal(_cat(grad), gh)                    # gradients untouched
    for rows in (grad, err, w):                              # nothing written outside the tensors
        for row in rows:
            for t in row:
                base = t.untyped_storage()
                full = torch.tensor([], dtype=torch.float32, device="cuda").set_(base)
                o = t.storage_offset()
                assert torch.isnan(full[:o]).all() and torch.isnan(full[o + t.numel():]).all()
    plan.destroy()
    ctx.destroy()


def test_segment_list_equals_flat_path_and_is_reproducible():
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 32)
    n, P = wl.n, wl.P
    flat_g = B.padded_rows(P, n, "cuda")
    W.fill_gradients(wl, 0, flat_g)
    flat_e = B.padded_rows(P, n, "cuda", fill=0.0)
    flat_w = torch.empty(n, device="cuda")
    W.init_weights(wl, flat_w)
    sizes = [s.numel for s in wl.segments]

    def split(row):
        return [t.clone() for t in torch.split(row, sizes)]

    outs = []
    for _ in range(2):
        grad = [split(flat_g[p]) for p in range(P)]
        err = [split(flat_e[p]) for p in range(P)]
        w = split(flat_w)
        ctx = B.a2sgd_create(n, P, 0, EF)
        plan = B.a2sgd_segments_create(ctx, grad, err, w)
        B.a2sgd_step_segments(ctx, plan, wl.lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        outs.append((lm.tobytes(), gm.tobytes(), cnt.tobytes(), torch.cat(w).cpu().numpy().tobytes(),
                     _cat(err).tobytes()))
        plan.destroy()
        ctx.destroy()
    assert outs[0] == outs[1]
    ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_TWO_PASS)
    B.a2sgd_step(ctx, flat_w, flat_g, flat_e, wl.lr)
    lm_f, gm_f, cnt_f, _ = B.a2sgd_read_stats(ctx)
    assert np.array_equal(cnt_f, cnt)
    assert_means(lm, lm_f)
    assert_means(gm, gm_f)
    assert_state(torch.cat(w).cpu().numpy(), flat_w.cpu().numpy(), _cat(err), flat_e.cpu().numpy(), gm_f, "flat vs segments")
    ctx.destroy()


def test_segment_plan_argument_checks():
    ctx = B.a2sgd_create(100, 2, 0, EF)
    g = [[torch.zeros(60, device="cuda"), torch.zeros(40, device="cuda")] for _ in range(2)]
    w = [torch.zeros(60, device="cuda"), torch.zeros(40, device="cuda")]
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_segments_create(ctx, g, None, w)                 # EF needs err
    assert ei.value.status == B.ERR_ARG
    bad = [[torch.zeros(60, device="cuda"), torch.zeros(41, device="cuda")] for _ in range(2)]
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_segments_create(ctx, bad, bad, w)                # sizes do not add up to n
    assert ei.value.status == B.ERR_ARG
    ctx.destroy()


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
def test_per_segment_learning_rates(mode, replicated):
    """Layer-wise learning rates (the hook for LARS): the means are whole-model, the update of
    each tensor uses its own rate.  Reference: the oracle's encode on the concatenation, then its
    decode tensor by tensor with that tensor's rate."""
    P = 4
    sizes = [5, 2048, 70_001, 33, 4096, 12_345]
    offsets = [0, 0, 1, 0]
    n = sum(sizes)
    gen = torch.Generator("cuda").manual_seed(77)
    grad = [_tensors(sizes, offsets, gen, 1e-3) for _ in range(P)]
    err = [_tensors(sizes, offsets, gen, 3e-4) for _ in range(P)]
    w = [_tensors(sizes, offsets, gen, 0.02) for _ in range(P if replicated else 1)]
    lrs = np.array([0.5, 0.01, 0.2, 1.0, 0.05, 0.125], np.float32)
    gh, eh = _cat(grad), _cat(err)
    wh = _cat(w) if replicated else _cat(w)[0]
    lm_ref, cnt_ref, _ = oracle.encode(gh, eh if mode == EF else None, mode=mode)
    gm_ref = oracle.global_average(lm_ref)
    off = 0
    for s, lr in zip(sizes, lrs):
        g_s = np.ascontiguousarray(gh[:, off:off + s])
        e_s = np.ascontiguousarray(eh[:, off:off + s])
        w_s = np.ascontiguousarray(wh[:, off:off + s]) if replicated else wh[off:off + s].copy()
        oracle.decode_update(w_s, g_s, e_s, lm_ref, gm_ref, float(lr), mode=mode)
        eh[:, off:off + s] = e_s
        if replicated:
            wh[:, off:off + s] = w_s
        else:
            wh[off:off + s] = w_s
        off += s
    ctx = B.a2sgd_create(n, P, 0, mode)
    plan = B.a2sgd_segments_create(ctx, grad, err, w if replicated else w[0], w_replicated=replicated)
    B.a2sgd_step_segments_lr(ctx, plan, torch.from_numpy(lrs).cuda())
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    w_got = _cat(w) if replicated else _cat(w)[0]
    assert_state(w_got, wh, _cat(err), eh, gm_ref, "per-segment lr")
    plan.destroy()
    ctx.destroy()


@pytest.mark.parametrize("mode", [EF, ALG1])
def test_staged_segment_calls_match_oracle(mode):
    """a2sgd_encode_segments -> a2sgd_global_average -> a2sgd_decode_update_segments, the three
    stages as separate calls on caller-owned means, against the oracle on the concatenation."""
    P = 3
    sizes = [2048, 5, 70_001, 4096, 999]
    n = sum(sizes)
    gen = torch.Generator("cuda").manual_seed(5)
    grad = [_tensors(sizes, [0, 1], gen, 1e-3) for _ in range(P)]
    err = [_tensors(sizes, [0, 1], gen, 3e-4) for _ in range(P)]
    w = _tensors(sizes, [0, 1], gen, 0.02)
    gh, eh, wh = _cat(grad), _cat(err), _cat([w])[0]
    ctx = B.a2sgd_create(n, P, 0, mode)
    plan = B.a2sgd_segments_create(ctx, grad, err, w)
    lm = torch.full((P + 2, 2), float("nan"), device="cuda")
    cnt = torch.zeros(P, dtype=torch.int64, device="cuda")
    gm = torch.zeros(2, device="cuda")
    B.a2sgd_encode_segments(ctx, plan, lm[1:P + 1], cnt)
    B.a2sgd_global_average(ctx, lm[1:P + 1], gm)
    B.a2sgd_decode_update_segments(ctx, plan, lm[1:P + 1], gm, 0.1)
    lm_ref, gm_ref, cnt_ref = oracle.step(wh, gh, eh, 0.1, mode=mode)
    assert np.array_equal(cnt.cpu().numpy().astype(np.uint64), cnt_ref)
    assert_means(lm[1:P + 1].cpu().numpy(), lm_ref)
    assert_means(gm.cpu().numpy(), gm_ref)
    assert torch.isnan(lm[0]).all() and torch.isnan(lm[P + 1]).all()      # two floats per worker, nothing else
    assert_state(_cat([w])[0], wh, _cat(err), eh, gm_ref, "staged segments")
    plan.destroy()
    ctx.destroy()


def test_thousands_of_tensors_take_the_tile_table_path():
    """More tensors than the decode kernel scans for (it then reads per-tile descriptors instead)."""
    P, S = 2, 4500
    rng = np.random.default_rng(9)
    sizes = [int(x) for x in rng.integers(1, 40, size=S)] + [5000]
    n = sum(sizes)
    gen = torch.Generator("cuda").manual_seed(11)
    flat_g = torch.empty((P, n), device="cuda").normal_(0, 1e-3, generator=gen)
    flat_e = torch.empty((P, n), device="cuda").normal_(0, 3e-4, generator=gen)
    flat_w = torch.empty(n, device="cuda").normal_(0, 0.02, generator=gen)
    gh, eh, wh = flat_g.cpu().numpy(), flat_e.cpu().numpy(), flat_w.cpu().numpy()
    grad = [list(torch.split(flat_g[p], sizes)) for p in range(P)]       # views at arbitrary 4-byte offsets
    err = [list(torch.split(flat_e[p], sizes)) for p in range(P)]
    w = list(torch.split(flat_w, sizes))
    ctx = B.a2sgd_create(n, P, 0, EF)
    plan = B.a2sgd_segments_create(ctx, grad, err, w)
    B.a2sgd_step_segments(ctx, plan, 0.1)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, gm_ref, cnt_ref = oracle.step(wh, gh, eh, 0.1, mode=oracle.MODE_EF)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    assert_state(flat_w.cpu().numpy(), wh, flat_e.cpu().numpy(), eh, gm_ref, "4501 tensors")
    plan.destroy()
    ctx.destroy()


def test_alg1_error_table_with_a_missing_entry_is_rejected():
    ctx = B.a2sgd_create(100, 2, 0, ALG1)
    g = [[torch.zeros(60, device="cuda"), torch.zeros(40, device="cuda")] for _ in range(2)]
    w = [torch.zeros(60, device="cuda"), torch.zeros(40, device="cuda")]
    import ctypes
    numel = (ctypes.c_uint64 * 2)(60, 40)
    vp = ctypes.c_void_p
    g_tab = (vp * 4)(*[t.data_ptr() for row in g for t in row])
    e_tab = (vp * 4)(g[0][0].data_ptr(), None, g[1][0].data_ptr(), g[1][1].data_ptr())   # one NULL entry
    w_tab = (vp * 2)(*[t.data_ptr() for t in w])
    out = vp()
    rc = B.lib().a2sgd_segments_create(ctx.handle, 2, numel, g_tab, e_tab, w_tab, 0, ctypes.byref(out))
    assert rc == B.ERR_ARG and not out
    ctx.destroy()


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,offsets", [(1, [0]), (4, [0]), (3, [0, 1, 0, 8, 3]), (8, [0, 0, 2])])
def test_per_tensor_means_variant_equals_one_oracle_step_per_tensor(mode, replicated, P, offsets):
    """a2sgd_step_segments_per_tensor compresses every tensor on its own: the reference is the
    oracle's step called once per tensor (its own local means, its own global means)."""
    sizes = [1, 5, 2047, 2048, 2049, 70_001, 33, 3 * 2048, 12_345, 64]
    S = len(sizes)
    gen = torch.Generator("cuda").manual_seed(31 * P + len(offsets))
    grad = [_tensors(sizes, offsets, gen, 1e-3) for _ in range(P)]
    for p in range(P):                      # a different scale per tensor, so per-tensor means really differ
        for k, t in enumerate(grad[p]):
            t.mul_(10.0 ** (k % 4))
    err = [_tensors(sizes, offsets, gen, 3e-4) for _ in range(P)]
    w = [_tensors(sizes, offsets, gen, 0.02) for _ in range(P if replicated else 1)]
    lrs = torch.tensor([0.1 * (1 + k % 3) for k in range(S)], device="cuda")
    # reference: one oracle step per tensor
    refs = []
    for k in range(S):
        g_k = np.stack([grad[p][k].cpu().numpy() for p in range(P)])
        e_k = np.stack([err[p][k].cpu().numpy() for p in range(P)])
        w_k = np.stack([w[p][k].cpu().numpy() for p in range(P)]) if replicated else w[0][k].cpu().numpy().copy()
        lm, gm, cnt = oracle.step(w_k, g_k, e_k, float(lrs[k]), mode=mode)
        refs.append((lm, gm, cnt, w_k, e_k))
    ctx = B.a2sgd_create(sum(sizes), P, 0, mode)
    plan = B.a2sgd_segments_create(ctx, grad, err, w if replicated else w[0], w_replicated=replicated)
    B.a2sgd_step_segments_per_tensor(ctx, plan, 0.0, lrs)
    lm_all, gm_all, cnt_all = B.a2sgd_read_segment_stats(ctx, plan, S)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    for k, (lm, gm, cnt, w_k, e_k) in enumerate(refs):
        assert np.array_equal(cnt_all[k], cnt), f"tensor {k} counts"
        assert_means(lm_all[k], lm, f"tensor {k} local means")
        assert_means(gm_all[k], gm, f"tensor {k} global means")
        w_got = np.stack([w[p][k].cpu().numpy() for p in range(P)]) if replicated else w[0][k].cpu().numpy()
        e_got = np.stack([err[p][k].cpu().numpy() for p in range(P)])
        assert_state(w_got, w_k, e_got, e_k, gm, f"tensor {k}")
    for rows in (grad, err, w):                              # nothing written outside the tensors
        for row in rows:
            for t in row:
                full = torch.tensor([], dtype=torch.float32, device="cuda").set_(t.untyped_storage())
                o = t.storage_offset()
                assert torch.isnan(full[:o]).all() and torch.isnan(full[o + t.numel():]).all()
    # a second step on the same plan reuses the scratch and stays reproducible
    B.a2sgd_step_segments_per_tensor(ctx, plan, 0.0, lrs)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    plan.destroy()
    ctx.destroy()


def test_per_tensor_variant_with_equal_tensors_matches_whole_model_step():
    """If every tensor holds the same values, per-tensor means equal whole-model means, so the two
    variants must produce the same weights (to rounding of the differently ordered sums)."""
    P, n_t, S = 2, 4096, 3
    gen = torch.Generator("cuda").manual_seed(8)
    g0 = [torch.empty(n_t, device="cuda").normal_(0, 1e-3, generator=gen) for _ in range(P)]
    outs = []
    for variant in ("whole", "per_tensor"):
        grad = [[g0[p].clone() for _ in range(S)] for p in range(P)]
        err = [[torch.zeros(n_t, device="cuda") for _ in range(S)] for _ in range(P)]
        w = [torch.ones(n_t, device="cuda") for _ in range(S)]
        ctx = B.a2sgd_create(n_t * S, P, 0, EF)
        plan = B.a2sgd_segments_create(ctx, grad, err, w)
        if variant == "whole":
            B.a2sgd_step_segments(ctx, plan, 0.1)
        else:
            B.a2sgd_step_segments_per_tensor(ctx, plan, 0.1)
        torch.cuda.synchronize()
        outs.append(torch.cat(w).cpu().numpy())
        plan.destroy()
        ctx.destroy()
    assert np.allclose(outs[0], outs[1], rtol=0, atol=1e-9)
