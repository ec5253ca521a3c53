"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from paper_2006_07405_b200 import workloads as W
from parity_util import assert_means, assert_state

pytestmark = pytest.mark.gpu

EF, ALG1 = B.MODE_EF, B.MODE_ALG1
NAN = float("nan")


def _state(seed, P, n, *, pad=0, off=(0, 0, 0), replicated=False, g_scale=1e-3, e_scale=3e-4):
    """Seeded g, e, w on the GPU inside NaN-filled guard bands.  ``off`` shifts the start of
    the g / e / w rows by that many elements (pointer misalignment); ``pad`` widens the row
    stride beyond n.  Returns the views the library sees plus the raw buffers."""
    rng = np.random.default_rng(seed)
    stride = n + pad
    raw = {}
    views = {}
    for k, (name, scale, rows, o) in enumerate([("g", g_scale, P, off[0]), ("e", e_scale, P, off[1]),
                                                ("w", 0.02, P if replicated else 1, off[2])]):
        buf = np.full(8 + o + rows * stride + 8, NAN, np.float32)
        vals = (rng.standard_normal((rows, n)) * scale).astype(np.float32)
        for r in range(rows):
            buf[8 + o + r * stride: 8 + o + r * stride + n] = vals[r]
        t = torch.from_numpy(buf).cuda()
        raw[name] = t
        v = t[8 + o: 8 + o + rows * stride].view(rows, stride)[:, :n]
        views[name] = v if (name != "w" or replicated) else v[0]
    return views, raw, stride


def _host(views):
    g = views["g"].cpu().numpy().copy()
    e = views["e"].cpu().numpy().copy()
    w = views["w"].cpu().numpy().copy()
    return g, e, w


def _guards_intact(raw, views, n, stride, rows_of):
    """Everything outside the n live elements of each row is still NaN."""
    for name, t in raw.items():
        buf = t.cpu().numpy()
        live = np.zeros(buf.shape, bool)
        v = views[name]
        start = (v.data_ptr() - t.data_ptr()) // 4
        for r in range(rows_of[name]):
            live[start + r * stride: start + r * stride + n] = True
        assert np.isnan(buf[~live]).all(), f"{name}: guard band overwritten"
        assert np.isfinite(buf[live]).all(), f"{name}: live element not finite"


SIZES = [1, 2, 3, 4, 5, 31, 32, 33, 127, 1023, 1024, 1025, 4099, 65536 + 7, (1 << 20) - 1, (1 << 20) + 1]


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("n", SIZES)
def test_single_step_matches_oracle(mode, replicated, n):
    P = [1, 2, 3, 4, 8, 16][(n + int(replicated)) % 6]
    # worker stride chosen so that all three kernel families are hit across the size list:
    # stride % 8 == 0 -> 256-bit kernels, stride % 8 == 4 -> 128-bit kernels, stride % 4 == 1 -> scalar
    want = [0, 4, 1][n % 3]
    pad = (want - n) % 8
    views, raw, stride = _state(1000 + n, P, n, pad=pad, replicated=replicated)
    g, e, w = _host(views)
    ctx = B.a2sgd_create(n, P, 0, mode | B.FORCE_TWO_PASS)
    # stage 1: encode (means, counts, mask) -- bit-exact integers, 1e-6 means
    lm_buf = torch.full((P + 2, 2), NAN, device="cuda")
    lm = lm_buf[1:P + 1]
    cnt = torch.zeros(P, dtype=torch.int64, device="cuda")
    words = (n + 31) // 32
    mask = torch.zeros((P, words), dtype=torch.int32, device="cuda")
    B.a2sgd_encode(ctx, views["g"], views["e"] if mode == EF else None, lm, cnt, mask)
    lm_ref, cnt_ref, mask_ref = oracle.encode(g, e if mode == EF else None, mode=mode, want_mask=True)
    assert np.array_equal(cnt.cpu().numpy().astype(np.uint64), cnt_ref)
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), mask_ref)
    assert_means(lm.cpu().numpy(), lm_ref, "local means")
    # payload: exactly two floats per worker were written
    assert torch.isnan(lm_buf[0]).all() and torch.isnan(lm_buf[P + 1]).all()
    # stage 2: global average
    gm = torch.zeros(2, device="cuda")
    B.a2sgd_global_average(ctx, lm, gm)
    gm_ref = oracle.global_average(lm_ref)
    assert_means(gm.cpu().numpy(), gm_ref, "global means")
    # stage 3: decode / residual / SGD on copies, against the oracle's full step
    w_staged = raw["w"].clone()
    e_staged = raw["e"].clone()
    w_view = w_staged[(views["w"].data_ptr() - raw["w"].data_ptr()) // 4:]
    e_view = e_staged[(views["e"].data_ptr() - raw["e"].data_ptr()) // 4:]
    w_arg = w_view[:P * stride].view(P, stride)[:, :n] if replicated else w_view[:n]
    e_arg = e_view[:P * stride].view(P, stride)[:, :n]
    B.a2sgd_decode_update(ctx, w_arg, views["g"], e_arg, lm, gm, 0.1)
    w_ref, e_ref = w.copy(), e.copy()
    lm_o, gm_o, cnt_o = oracle.step(w_ref, g, e_ref, 0.1, mode=mode)
    assert_state(w_arg.cpu().numpy(), w_ref, e_arg.cpu().numpy(), e_ref, gm_o, f"staged n={n} P={P}")
    # default context (takes the single-launch path when n*P fits on chip) on second copies
    ctx2 = B.a2sgd_create(n, P, 0, mode)
    w2_raw, e2_raw = raw["w"].clone(), raw["e"].clone()
    w2_view = w2_raw[(views["w"].data_ptr() - raw["w"].data_ptr()) // 4:]
    e2_view = e2_raw[(views["e"].data_ptr() - raw["e"].data_ptr()) // 4:]
    w2 = w2_view[:P * stride].view(P, stride)[:, :n] if replicated else w2_view[:n]
    e2 = e2_view[:P * stride].view(P, stride)[:, :n]
    B.a2sgd_step(ctx2, w2, views["g"], e2, 0.1)
    lm_c, gm_c, cnt_c, status = B.a2sgd_read_stats(ctx2)
    assert status == B.OK and np.array_equal(cnt_c, cnt_ref)
    assert_means(lm_c, lm_ref, "default step local means")
    assert_means(gm_c, gm_ref, "default step global means")
    assert_state(w2.cpu().numpy(), w_ref, e2.cpu().numpy(), e_ref, gm_o, f"default step n={n} P={P}")
    raw2 = {"g": raw["g"], "e": e2_raw, "w": w2_raw}
    views2 = {"g": views["g"], "e": e2, "w": w2}
    _guards_intact(raw2, views2, n, stride, {"g": P, "e": P, "w": P if replicated else 1})
    ctx2.destroy()
    # fused two-pass step on the originals: same bits as the staged calls
    B.a2sgd_step(ctx, views["w"], views["g"], views["e"], 0.1)
    lm_s, gm_s, cnt_s, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    assert np.array_equal(cnt_s, cnt_ref)
    assert np.array_equal(lm_s, lm.cpu().numpy()) and np.array_equal(gm_s, gm.cpu().numpy())
    assert torch.equal(views["w"], w_arg) and torch.equal(views["e"], e_arg)
    rows = {"g": P, "e": P, "w": P if replicated else 1}
    _guards_intact(raw, views, n, stride, rows)
    # the gradient is never written
    assert np.array_equal(views["g"].cpu().numpy(), g)
    ctx.destroy()


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("off", [(1, 0, 0), (0, 1, 0), (0, 0, 1), (1, 2, 3), (3, 3, 3), (2, 0, 2)])
def test_misaligned_pointers(mode, off):
    n, P = 10007, 3
    for replicated in (False, True):
        views, raw, stride = _state(77, P, n, pad=3, off=off, replicated=replicated)
        g, e, w = _host(views)
        ctx = B.a2sgd_create(n, P, 0, mode)
        B.a2sgd_step(ctx, views["w"], views["g"], views["e"], 0.05)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        lm_ref, gm_ref, cnt_ref = oracle.step(w, g, e, 0.05, mode=mode)
        assert status == B.OK and np.array_equal(cnt, cnt_ref)
        assert_means(lm, lm_ref)
        assert_means(gm, gm_ref)
        assert_state(views["w"].cpu().numpy(), w, views["e"].cpu().numpy(), e, gm_ref, f"off={off}")
        _guards_intact(raw, views, n, stride, {"g": P, "e": P, "w": P if replicated else 1})
        ctx.destroy()


def test_alg1_without_error_buffer_and_single_worker_is_dense_sgd():
    n = 50001
    views, raw, stride = _state(5, 1, n)
    g, e, w = _host(views)
    ctx = B.a2sgd_create(n, 1, 0, ALG1)
    B.a2sgd_step(ctx, views["w"], views["g"], None, 0.1)
    torch.cuda.synchronize()
    # P = 1: Algorithm 1 returns g itself, the update is one fp32 fma per element
    ref = w.astype(np.float64) - np.float64(np.float32(0.1)) * g[0].astype(np.float64)
    got = views["w"].cpu().numpy()
    assert np.max(np.abs(got - ref)) <= np.spacing(np.abs(w).max())
    assert np.array_equal(views["e"].cpu().numpy(), e)   # untouched when no err pointer is passed
    ctx.destroy()


@pytest.mark.parametrize("case", ["all_pos", "all_neg", "zeros", "neg_zero", "subnormal", "two_valued"])
def test_degenerate_inputs(case):
    n, P = 3001, 2
    views, raw, stride = _state(9, P, n)
    g = views["g"]
    views["e"].zero_()
    if case == "all_pos":
        g.abs_()
    elif case == "all_neg":
        g.abs_().neg_().sub_(1e-9)
    elif case == "zeros":
        g.zero_()
    elif case == "neg_zero":
        g.zero_().neg_()
    elif case == "subnormal":
        g.copy_(torch.where(g >= 0, torch.full_like(g, 1e-45), torch.full_like(g, -1e-45)))
    elif case == "two_valued":
        g.copy_(torch.where(g >= 0, torch.full_like(g, 0.75), torch.full_like(g, -0.125)))
    gh, eh, wh = _host(views)
    ctx = B.a2sgd_create(n, P, 0, EF)
    lm = torch.zeros((P, 2), device="cuda")
    cnt = torch.zeros(P, dtype=torch.int64, device="cuda")
    mask = torch.zeros((P, (n + 31) // 32), dtype=torch.int32, device="cuda")
    B.a2sgd_encode(ctx, views["g"], views["e"], lm, cnt, mask)
    lm_ref, cnt_ref, mask_ref = oracle.encode(gh, eh, mode=EF, want_mask=True)
    assert np.array_equal(cnt.cpu().numpy().astype(np.uint64), cnt_ref)
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), mask_ref)
    if case in ("all_pos", "all_neg"):
        assert_means(lm.cpu().numpy(), lm_ref)
    else:
        assert np.array_equal(lm.cpu().numpy(), lm_ref)  # sums of these values are exact in fp32
    B.a2sgd_step(ctx, views["w"], views["g"], views["e"], 0.1)
    oracle.step(wh, gh, eh, 0.1, mode=EF)
    _, gm, _, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    assert_state(views["w"].cpu().numpy(), wh, views["e"].cpu().numpy(), eh, gm, case)
    if case == "two_valued":
        assert not views["e"].any()
    ctx.destroy()


def test_run_to_run_bitwise_reproducible():
    wl = W.scaled(W.get_workload("c3_resnet50"), 8)
    n, P = wl.n, wl.P
    g = torch.empty((P, n), device="cuda")
    W.fill_gradients(wl, 0, g)
    e0 = torch.randn((P, n), device="cuda", generator=torch.Generator("cuda").manual_seed(3)) * 1e-4
    w0 = torch.empty(n, device="cuda")
    W.init_weights(wl, w0)
    outs = []
    for _ in range(3):
        ctx = B.a2sgd_create(n, P, 0, EF)
        e, w = e0.clone(), w0.clone()
        B.a2sgd_step(ctx, w, g, e, wl.lr)
        lm, gm, cnt, _ = B.a2sgd_read_stats(ctx)
        outs.append((lm.tobytes(), gm.tobytes(), cnt.tobytes(), e.cpu().numpy().tobytes(), w.cpu().numpy().tobytes()))
        ctx.destroy()
    assert outs[0] == outs[1] == outs[2]


@pytest.mark.parametrize("name,div", [("c1_flat_1m", 1), ("c2_lstm_ptb", 16), ("c3_resnet50", 4),
                                      ("c4_vgg16", 32), ("c5_gpt2_xl", 256)])
@pytest.mark.parametrize("mode", [EF, ALG1])
def test_free_running_multi_step(name, div, mode):
    """The benchmark configurations (tensor structure kept, lengths divided so that the oracle
    finishes in seconds), run for their stated number of steps, GPU and oracle each on its own
    evolving state."""
    wl = W.get_workload(name)
    wl = W.scaled(wl, div) if div > 1 else wl
    n, P = wl.n, wl.P
    g = torch.empty((P, n), device="cuda")
    e = torch.zeros((P, n), device="cuda")
    w = torch.empty(n, device="cuda")
    W.init_weights(wl, w)
    e_ref = np.zeros((P, n), np.float32)
    w_ref = w.cpu().numpy().copy()
    ctx = B.a2sgd_create(n, P, 0, mode)
    flips = 0
    for step in range(wl.steps):
        W.fill_gradients(wl, step, g)
        gh = g.cpu().numpy()
        B.a2sgd_step(ctx, w, g, e, wl.lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        lm_ref, gm_ref, cnt_ref = oracle.step(w_ref, gh, e_ref, wl.lr, mode=mode)
        assert status == B.OK
        # from step 2 on the two error buffers differ by rounding, so an element whose
        # compensated value sits at rounding level may change group: count, do not fail
        flips += int(np.abs(cnt.astype(np.int64) - cnt_ref.astype(np.int64)).sum())
        if step == 0:
            assert np.array_equal(cnt, cnt_ref)
        assert_means(lm, lm_ref, f"{name} step {step} local means")
        assert_means(gm, gm_ref, f"{name} step {step} global means")
        allowed = 0 if step == 0 else max(2, n * P // 1_000_000)
        assert_state(w.cpu().numpy(), w_ref, e.cpu().numpy(), e_ref, gm_ref, f"{name} step {step}",
                     max_outliers=allowed)
    assert flips <= max(2, n * P // 1_000_000), f"{flips} group changes"
    ctx.destroy()


def test_nonfinite_input_is_latched_in_status_word():
    n, P = 5000, 2
    views, raw, stride = _state(21, P, n)
    views["g"][1, 1234] = float("inf")
    ctx = B.a2sgd_create(n, P, 0, EF)
    lm = torch.zeros((P, 2), device="cuda")
    B.a2sgd_encode(ctx, views["g"], views["e"], lm)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.ERR_NONFINITE
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK          # the latch is cleared by the read
    ctx.destroy()


def test_bad_arguments_return_status_and_launch_nothing():
    n, P = 1000, 2
    views, raw, stride = _state(22, P, n)
    before = {k: v.clone() for k, v in raw.items()}
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_create(0, 1)
    assert ei.value.status == B.ERR_ARG
    with pytest.raises(B.A2SGDError):
        B.a2sgd_create(10, 0)
    with pytest.raises(B.A2SGDError):
        B.a2sgd_create(10, 1025)
    with pytest.raises(B.A2SGDError):
        B.a2sgd_create(10, 1, 0, 1 << 20)
    with pytest.raises(B.A2SGDError):
        B.a2sgd_create(10, 1, 99)
    ctx = B.a2sgd_create(n, P, 0, EF)
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_step(ctx, views["w"], views["g"], None, 0.1)       # EF needs err
    assert ei.value.status == B.ERR_ARG
    with pytest.raises(B.A2SGDError) as ei:                          # worker stride < n
        B.a2sgd_step(ctx, views["w"], views["g"][:, : n // 2].contiguous().view(P, n // 2), views["e"], 0.1)
    assert ei.value.status == B.ERR_ARG
    h = ctx.handle
    st = B.lib().a2sgd_step(h, views["w"].data_ptr() + 2, 0, views["g"].data_ptr(), stride,
                            views["e"].data_ptr(), stride, 0.1, None)
    assert st == B.ERR_ALIGN
    torch.cuda.synchronize()
    for k in raw:
        assert torch.equal(torch.nan_to_num(raw[k]), torch.nan_to_num(before[k]))
    assert "argument" in B.status_string(B.ERR_ARG)
    ctx.destroy()


def test_checkpoint_resume_is_bitwise():
    """All state is caller-owned: 5 steps == 3 steps, copy out / in, new context, 2 steps."""
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 64)
    n, P = wl.n, wl.P
    g = torch.empty((P, n), device="cuda")

    def run(split):
        e = torch.zeros((P, n), device="cuda")
        w = torch.empty(n, device="cuda")
        W.init_weights(wl, w)
        ctx = B.a2sgd_create(n, P, 0, EF)
        for step in range(5):
            if step == split:
                e = e.cpu().cuda()
                w = w.cpu().cuda()
                ctx.destroy()
                ctx = B.a2sgd_create(n, P, 0, EF)
            W.fill_gradients(wl, step, g)
            B.a2sgd_step(ctx, w, g, e, wl.lr)
        torch.cuda.synchronize()
        return e.cpu(), w.cpu()

    ea, wa = run(None)
    eb, wb = run(3)
    assert torch.equal(ea, eb) and torch.equal(wa, wb)


def test_host_gradient_entry_point():
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 32)
    n, P = wl.n, wl.P
    g_host = torch.empty((P, n)).pin_memory()
    W.fill_gradients(wl, 0, g_host)
    staging = torch.empty((P, n), device="cuda")
    e = torch.zeros((P, n), device="cuda")
    w = torch.empty(n, device="cuda")
    W.init_weights(wl, w)
    w_ref = w.cpu().numpy().copy()
    e_ref = np.zeros((P, n), np.float32)
    means = torch.zeros(2 * P + 2).pin_memory()
    ctx = B.a2sgd_create(n, P, 0, EF)
    B.a2sgd_step_host(ctx, w, g_host, staging, e, wl.lr, means)
    lm_ref, gm_ref, _ = oracle.step(w_ref, g_host.numpy(), e_ref, wl.lr, mode=EF)
    assert_means(means[:2 * P].numpy().reshape(P, 2), lm_ref)
    assert_means(means[2 * P:].numpy(), gm_ref)
    assert_state(w.cpu().numpy(), w_ref, e.cpu().numpy(), e_ref, gm_ref, "host entry")
    ctx.destroy()


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("P,n", [(1, 1 << 20), (1, (1 << 20) + 3), (2, 500_001), (4, 250_000), (8, 123_457), (4, 5),
                                 # beyond the register-resident capacity: the L2-resident form
                                 (1, 5_000_003), (2, 2_500_001), (4, 1_200_000), (8, 400_002)])
@pytest.mark.parametrize("replicated", [False, True])
def test_single_launch_path(mode, P, n, replicated):
    """The cooperative single-launch kernel (v kept in registers between the two phases) against
    the oracle, and forced explicitly so that a silent fall-back to two launches cannot pass."""
    g = B.padded_rows(P, n, "cuda")
    e = B.padded_rows(P, n, "cuda")
    gen = torch.Generator("cuda").manual_seed(n + P)
    g.normal_(0.0, 1e-3, generator=gen)
    e.normal_(0.0, 3e-4, generator=gen)
    w = B.padded_rows(P, n, "cuda") if replicated else torch.empty(n, device="cuda")
    w.normal_(0.0, 0.02, generator=gen)
    gh, eh, wh = g.cpu().numpy().copy(), e.cpu().numpy().copy(), w.cpu().numpy().copy()
    ctx = B.a2sgd_create(n, P, 0, mode | B.FORCE_COOPERATIVE)
    assert B.a2sgd_launch_info(ctx, shared_w=not replicated)["single_launch"]
    outs = []
    for rep in range(2):                     # twice from the same state: bitwise reproducible
        w_i, e_i = w.clone(), e.clone()
        if replicated:
            w_i = B.padded_rows(P, n, "cuda"); w_i.copy_(w)
        e_pad = B.padded_rows(P, n, "cuda"); e_pad.copy_(e); e_i = e_pad
        B.a2sgd_step(ctx, w_i, g, e_i, 0.1)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        outs.append((lm.tobytes(), gm.tobytes(), cnt.tobytes(), w_i.cpu().numpy().tobytes(), e_i.cpu().numpy().tobytes()))
    assert outs[0] == outs[1]
    lm_ref, gm_ref, cnt_ref = oracle.step(wh, gh, eh, 0.1, mode=mode)
    assert np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    assert_state(w_i.cpu().numpy(), wh, e_i.cpu().numpy(), eh, gm_ref, f"coop P={P} n={n}")
    ctx.destroy()


def test_single_launch_path_refuses_what_does_not_fit():
    n, P = 1 << 24, 4
    g = torch.zeros((P, n), device="cuda")
    e = torch.zeros((P, n), device="cuda")
    w = torch.zeros(n, device="cuda")
    ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_COOPERATIVE)
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_step(ctx, w, g, e, 0.1)
    assert ei.value.status == B.ERR_TOO_LARGE
    ctx.destroy()
    ctx = B.a2sgd_create(1000, 3, 0, EF | B.FORCE_COOPERATIVE)     # P = 3 has no single-launch kernel
    with pytest.raises(B.A2SGDError):
        B.a2sgd_step(ctx, w[:1000], g[:3, :1000], e[:3, :1000], 0.1)
    ctx.destroy()


def test_bounded_barrier_wait_times_out_cleanly():
    """A grid barrier that can never open (the test hook asks for one arrival more than the
    grid has): every CTA gives up after its poll limit, nothing is written, the status word
    reports the timeout, and the device stays usable."""
    n, P = 200_000, 2
    g = B.padded_rows(P, n, "cuda"); g.normal_(0.0, 1e-3)
    e = B.padded_rows(P, n, "cuda"); e.normal_(0.0, 1e-4)
    w = torch.randn(n, device="cuda") * 0.02
    e0, w0 = e.clone(), w.clone()
    ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_COOPERATIVE | B.TEST_BARRIER_NEVER_OPENS)
    B.a2sgd_step(ctx, w, g, e, 0.1)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.ERR_TIMEOUT
    assert torch.equal(e, e0) and torch.equal(w, w0)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    ctx.destroy()
    good = B.a2sgd_create(n, P, 0, EF | B.FORCE_COOPERATIVE)
    B.a2sgd_step(good, w, g, e, 0.1)
    *_, status = B.a2sgd_read_stats(good)
    assert status == B.OK and not torch.equal(w, w0)
    good.destroy()


@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,n,pad", [(1, 1, 0), (2, 7, 1), (3, 1000, 0), (4, 65536 + 5, 3), (4, 1 << 20, 0),
                                     (8, 300_001, 7), (5, 123_456, 0), (16, 4099, 1)])
def test_dense_sync_step_matches_oracle(replicated, P, n, pad):
    """Algorithm 1 lines 9-10: the dense averaging step that follows the compressed iterations."""
    views, raw, stride = _state(4000 + n, P, n, pad=pad, replicated=replicated, g_scale=1e-2)
    g, e, w = _host(views)
    ctx = B.a2sgd_create(n, P, 0, EF)
    B.a2sgd_dense_sync(ctx, views["w"], views["g"], 0.25)
    torch.cuda.synchronize()
    oracle.dense_sync(w, g, 0.25)
    got = views["w"].cpu().numpy()
    from parity_util import count_outliers, tau_w
    assert count_outliers(got, w, tau_w(w)) == 0
    # stricter: an fp32 sum of P terms and one fma against an fp64 reference
    bound = (P + 2) * np.spacing(np.float32(max(np.abs(w).max(), 0.25 * np.abs(g).max())))
    assert np.max(np.abs(got.astype(np.float64) - w.astype(np.float64))) <= bound
    assert np.array_equal(views["g"].cpu().numpy(), g) and np.array_equal(views["e"].cpu().numpy(), e)
    _guards_intact(raw, views, n, stride, {"g": P, "e": P, "w": P if replicated else 1})
    ctx.destroy()


def test_compressed_iterations_then_dense_sync_like_algorithm_1():
    """T-1 compressed iterations followed by the dense step, replicas as in Algorithm 1."""
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 64)
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, "cuda")
    w = B.padded_rows(P, n, "cuda")
    w0 = torch.empty(n, device="cuda")
    W.init_weights(wl, w0)
    w.copy_(w0.expand(P, n))
    w_ref = w.cpu().numpy().copy()
    ctx = B.a2sgd_create(n, P, 0, ALG1)
    for step in range(3):
        W.fill_gradients(wl, step, g)
        B.a2sgd_step(ctx, w, g, None, wl.lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        oracle.step(w_ref, g.cpu().numpy(), None, wl.lr, mode=ALG1)
    W.fill_gradients(wl, 3, g)
    B.a2sgd_dense_sync(ctx, w, g, wl.lr)
    oracle.dense_sync(w_ref, g.cpu().numpy(), wl.lr)
    from parity_util import count_outliers, tau_w
    assert count_outliers(w.cpu().numpy(), w_ref, tau_w(w_ref)) == 0
    ctx.destroy()


def _widen_bf16(t):
    """bfloat16 -> fp32 by the definition of the format (upper 16 bits of an fp32), in numpy."""
    u16 = t.view(torch.int16).cpu().numpy().view(np.uint16)
    return (u16.astype(np.uint32) << 16).view(np.float32)


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,n,stride_pad,off", [(1, 9, 0, 0), (4, 1 << 20, 0, 0), (4, 100_003, 5, 0), (3, 70_000, 0, 0),
                                                (8, 33_333, 3, 1), (2, 4096, 0, 3), (16, 2051, 13, 0)])
def test_bf16_gradient_step_matches_oracle_on_widened_gradients(mode, replicated, P, n, stride_pad, off):
    gen = torch.Generator("cuda").manual_seed(n + P)
    stride = n + stride_pad
    gbuf = torch.zeros(off + P * stride + 8, device="cuda")
    gbuf.normal_(0.0, 1e-3, generator=gen)
    g16_all = gbuf.to(torch.bfloat16)
    g16 = g16_all[off:off + P * stride].view(P, stride)[:, :n]
    assert np.array_equal(_widen_bf16(g16.contiguous()), g16.float().cpu().numpy())   # widening is exact
    e = torch.empty((P, stride), device="cuda")[:, :n]
    e.normal_(0.0, 3e-4, generator=gen)
    w = (torch.empty((P, stride), device="cuda")[:, :n] if replicated else torch.empty(n, device="cuda"))
    w.normal_(0.0, 0.02, generator=gen)
    gh = _widen_bf16(g16.contiguous()).reshape(P, n)
    eh, wh = e.cpu().numpy().copy(), w.cpu().numpy().copy()
    ctx = B.a2sgd_create(n, P, 0, mode)
    B.a2sgd_step_bf16(ctx, w, g16, e, 0.1)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, gm_ref, cnt_ref = oracle.step(wh, gh, eh, 0.1, mode=mode)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    assert_state(w.cpu().numpy(), wh, e.cpu().numpy(), eh, gm_ref, f"bf16 P={P} n={n}")
    assert torch.equal(g16_all, gbuf.to(torch.bfloat16))      # gradients untouched
    ctx.destroy()


def test_maximum_worker_count():
    """P = 1024 (the documented maximum): run-time-P kernels, one or two CTAs per worker in K1."""
    P, n = 1024, 3001
    views, raw, stride = _state(31, P, n, pad=3)
    g, e, w = _host(views)
    ctx = B.a2sgd_create(n, P, 0, EF)
    B.a2sgd_step(ctx, views["w"], views["g"], views["e"], 0.1)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, gm_ref, cnt_ref = oracle.step(w, g, e, 0.1, mode=EF)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    assert_state(views["w"].cpu().numpy(), w, views["e"].cpu().numpy(), e, gm_ref, "P=1024")
    _guards_intact(raw, views, n, stride, {"g": P, "e": P, "w": 1})
    ctx.destroy()


def test_randomised_shapes_strides_alignments():
    """Seeded random sweep over n, P, mode, weight layout, row stride and pointer offsets."""
    rng = np.random.default_rng(20060740)
    for trial in range(40):
        P = int(rng.choice([1, 2, 3, 4, 5, 8, 11, 16]))
        n = int(rng.choice([rng.integers(1, 300), rng.integers(300, 70_000), rng.integers(70_000, 400_000)]))
        mode = int(rng.choice([EF, ALG1]))
        replicated = bool(rng.integers(0, 2))
        pad = int(rng.choice([0, 0, (-n) % 8, (-n) % 32, rng.integers(0, 40)]))
        off = tuple(int(x) for x in rng.choice([0, 0, 0, 1, 2, 3, 4, 8], size=3))
        views, raw, stride = _state(5000 + trial, P, n, pad=pad, off=off, replicated=replicated,
                                    g_scale=float(10.0 ** rng.uniform(-5, 0)), e_scale=float(10.0 ** rng.uniform(-6, -1)))
        g, e, w = _host(views)
        ctx = B.a2sgd_create(n, P, 0, mode)
        lr = float(rng.choice([0.01, 0.1, 1.0]))
        B.a2sgd_step(ctx, views["w"], views["g"], views["e"], lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        lm_ref, gm_ref, cnt_ref = oracle.step(w, g, e, lr, mode=mode)
        what = f"trial {trial}: P={P} n={n} mode={mode} repl={replicated} pad={pad} off={off}"
        assert status == B.OK and np.array_equal(cnt, cnt_ref), what
        assert_means(lm, lm_ref, what)
        assert_means(gm, gm_ref, what)
        assert_state(views["w"].cpu().numpy(), w, views["e"].cpu().numpy(), e, gm_ref, what)
        _guards_intact(raw, views, n, stride, {"g": P, "e": P, "w": P if replicated else 1})
        ctx.destroy()


def test_steps_captured_in_a_cuda_graph_replay_bitwise():
    """The two launches of a step (programmatic dependent launch included) can be captured and
    replayed; replays give the same bits as eager launches."""
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 16)
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, "cuda")
    W.fill_gradients(wl, 0, g)
    w0 = torch.empty(n, device="cuda")
    W.init_weights(wl, w0)

    def run(use_graph):
        e = B.padded_rows(P, n, "cuda", fill=0.0)
        w = w0.clone()
        ctx = B.a2sgd_create(n, P, 0, EF)
        B.a2sgd_step(ctx, w, g, e, wl.lr)                     # warm-up outside any capture
        if use_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for _ in range(2):
                        B.a2sgd_step(ctx, w, g, e, wl.lr, stream=side)
            torch.cuda.current_stream().wait_stream(side)
            graph.replay()
            graph.replay()
        else:
            for _ in range(4):
                B.a2sgd_step(ctx, w, g, e, wl.lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        out = (status, lm.tobytes(), gm.tobytes(), cnt.tobytes(), w.cpu().numpy().tobytes(), e.cpu().numpy().tobytes())
        ctx.destroy()
        return out

    eager, replayed = run(False), run(True)
    assert eager[0] == B.OK and eager == replayed


def test_two_contexts_on_two_streams_do_not_interfere():
    wl = W.scaled(W.get_workload("c4_vgg16"), 32)
    n, P = wl.n, wl.P
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    states, refs = [], []
    for k in range(2):
        g = B.padded_rows(P, n, "cuda")
        W.fill_gradients(wl, k, g)
        e = B.padded_rows(P, n, "cuda", fill=0.0)
        w = torch.empty(n, device="cuda")
        W.init_weights(wl, w)
        states.append((g, e, w, B.a2sgd_create(n, P, 0, EF)))
        gh, eh, wh = g.cpu().numpy(), e.cpu().numpy().copy(), w.cpu().numpy().copy()
        for _ in range(3):
            oracle.step(wh, gh, eh, wl.lr, mode=EF)
        refs.append((eh, wh))
    torch.cuda.synchronize()
    for it in range(3):
        for k in range(2):
            g, e, w, ctx = states[k]
            with torch.cuda.stream(streams[k]):
                B.a2sgd_step(ctx, w, g, e, wl.lr, stream=streams[k])
    torch.cuda.synchronize()
    for k in range(2):
        g, e, w, ctx = states[k]
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        assert_state(w.cpu().numpy(), refs[k][1], e.cpu().numpy(), refs[k][0], gm, f"stream {k}", max_outliers=2)
        ctx.destroy()


def test_single_launch_step_replayed_from_a_one_step_graph():
    """A graph holding ONE cooperative step, replayed several times: the grid barrier must not
    depend on anything fixed at capture time."""
    n, P = 300_000, 1
    gen = torch.Generator("cuda").manual_seed(5)
    g = B.padded_rows(P, n, "cuda"); g.normal_(0.0, 1e-3, generator=gen)
    e0 = B.padded_rows(P, n, "cuda"); e0.normal_(0.0, 1e-4, generator=gen)
    w0 = torch.randn(n, device="cuda", generator=gen) * 0.02

    def run(use_graph):
        e = B.padded_rows(P, n, "cuda"); e.copy_(e0)
        w = w0.clone()
        ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_COOPERATIVE)
        B.a2sgd_step(ctx, w, g, e, 0.1)
        if use_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    B.a2sgd_step(ctx, w, g, e, 0.1, stream=side)
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(4):
                graph.replay()
        else:
            for _ in range(4):
                B.a2sgd_step(ctx, w, g, e, 0.1)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        out = (status, lm.tobytes(), gm.tobytes(), cnt.tobytes(), w.cpu().numpy().tobytes(), e.cpu().numpy().tobytes())
        ctx.destroy()
        return out

    eager, replayed = run(False), run(True)
    assert eager[0] == B.OK and eager == replayed


def test_pointer_check_flag_rejects_host_memory_before_any_launch():
    """With A2SGD_CHECK_POINTERS a host address is refused on the host; nothing reaches the GPU."""
    n, P = 4096, 2
    g = B.padded_rows(P, n, "cuda", 0.0)
    e = B.padded_rows(P, n, "cuda", 0.0)
    w = torch.zeros(n, device="cuda")
    host = np.zeros((P, n), np.float32)
    ctx = B.a2sgd_create(n, P, 0, EF | B.CHECK_POINTERS)
    h = ctx.handle
    lib = B.lib()
    assert lib.a2sgd_step(h, w.data_ptr(), 0, host.ctypes.data, n, e.data_ptr(), e.stride(0), 0.1, None) == B.ERR_ARG
    assert lib.a2sgd_step(h, host.ctypes.data, 0, g.data_ptr(), g.stride(0), e.data_ptr(), e.stride(0), 0.1, None) == B.ERR_ARG
    assert lib.a2sgd_dense_sync(h, w.data_ptr(), 0, host.ctypes.data, n, 0.1, None) == B.ERR_ARG
    B.a2sgd_step(ctx, w, g, e, 0.1)                          # device buffers pass
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    ctx.destroy()


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,n,stride_pad,off", [(1, 9, 0, 0), (4, 1 << 20, 0, 0), (4, 100_003, 5, 0), (8, 33_333, 3, 1)])
def test_f16_gradient_step_matches_oracle_on_widened_gradients(mode, replicated, P, n, stride_pad, off):
    gen = torch.Generator("cuda").manual_seed(n + 3 * P)
    stride = n + stride_pad
    gbuf = torch.zeros(off + P * stride + 8, device="cuda")
    gbuf.normal_(0.0, 1e-3, generator=gen)
    gbuf[::7] *= 1e-4                                       # some values in the half-precision subnormal range
    g16_all = gbuf.to(torch.float16)
    g16 = g16_all[off:off + P * stride].view(P, stride)[:, :n]
    # half -> fp32 by numpy's own conversion (exact): the oracle sees the widened values
    gh = g16.contiguous().view(torch.int16).cpu().numpy().view(np.float16).astype(np.float32).reshape(P, n)
    assert np.array_equal(gh, g16.float().cpu().numpy())
    e = torch.empty((P, stride), device="cuda")[:, :n]
    e.normal_(0.0, 3e-4, generator=gen)
    w = (torch.empty((P, stride), device="cuda")[:, :n] if replicated else torch.empty(n, device="cuda"))
    w.normal_(0.0, 0.02, generator=gen)
    eh, wh = e.cpu().numpy().copy(), w.cpu().numpy().copy()
    ctx = B.a2sgd_create(n, P, 0, mode)
    B.a2sgd_step_f16(ctx, w, g16, e, 0.1)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    lm_ref, gm_ref, cnt_ref = oracle.step(wh, gh, eh, 0.1, mode=mode)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    assert_state(w.cpu().numpy(), wh, e.cpu().numpy(), eh, gm_ref, f"f16 P={P} n={n}")
    ctx.destroy()


def test_average_from_allreduced_sums_matches_oracle():
    """Algorithm 1 line 5 in its all-reduce form: the collective delivers fp64 sums of the pairs,
    the library divides.  Reference: the oracle's global average of the same pairs."""
    rng = np.random.default_rng(4)
    for W_ in (1, 2, 3, 8, 64):
        lm = (rng.random((W_, 2)) * 1e-3).astype(np.float32)
        sums = torch.from_numpy(lm.astype(np.float64).sum(0)).cuda()      # what an all-reduce(SUM) returns
        ctx = B.a2sgd_create(1000, 1, 0, EF)
        gm = torch.zeros(2, device="cuda")
        B.a2sgd_global_average_from_sums(ctx, sums, W_, gm)
        assert_means(gm.cpu().numpy(), oracle.global_average(lm))
        ctx.destroy()


def test_dense_sync_on_an_allreduced_sum_matches_oracle():
    """Algorithm 1 lines 9-10 with one worker per GPU: the all-reduced SUM of the gradients goes in,
    the library divides by the worker count."""
    rng = np.random.default_rng(6)
    n, W_ = 100_003, 4
    g = (rng.standard_normal((W_, n)) * 1e-3).astype(np.float32)
    w0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    g_sum = torch.from_numpy(g).cuda().sum(0)                               # fp32 sum, as NCCL would form it
    w = torch.from_numpy(w0).cuda()
    ctx = B.a2sgd_create(n, 1, 0, EF)
    B.a2sgd_dense_sync_reduced(ctx, w, g_sum, W_, 0.1)
    w_ref = w0.copy()
    oracle.dense_sync(w_ref, g, 0.1)
    assert_state(w.cpu().numpy(), w_ref, None, None, None, "dense sync on a reduced sum")
    with pytest.raises(B.A2SGDError):                                       # contexts of one worker only
        ctx4 = B.a2sgd_create(n, 4, 0, EF)
        B.a2sgd_dense_sync_reduced(ctx4, w, g_sum, W_, 0.1)
    ctx.destroy()


def test_pointer_check_flag_covers_the_other_entry_points():
    """A2SGD_CHECK_POINTERS on the momentum, 16-bit-gradient, staged, reduced-sum and segment-list
    calls: a host address comes back as A2SGD_ERR_ARG before anything is launched."""
    import ctypes
    n, P = 4096, 2
    g = B.padded_rows(P, n, "cuda", 0.0)
    e = B.padded_rows(P, n, "cuda", 0.0)
    w = torch.zeros(n, device="cuda")
    m = torch.zeros(n, device="cuda")
    lm = torch.zeros((P, 2), device="cuda")
    gm = torch.zeros(2, device="cuda")
    host = np.zeros((P, n), np.float32)
    hp = host.ctypes.data
    ctx = B.a2sgd_create(n, P, 0, EF | B.CHECK_POINTERS)
    h, lib, s = ctx.handle, B.lib(), g.stride(0)
    assert lib.a2sgd_step_momentum(h, w.data_ptr(), 0, hp, 0, g.data_ptr(), s, e.data_ptr(), s, 0.1, 0.9, 0.0, None) == B.ERR_ARG
    assert lib.a2sgd_step_bf16(h, w.data_ptr(), 0, hp, n, e.data_ptr(), s, 0.1, None) == B.ERR_ARG
    assert lib.a2sgd_global_average(h, hp, gm.data_ptr(), None) == B.ERR_ARG
    assert lib.a2sgd_global_average_from_sums(h, hp, 2, gm.data_ptr(), None) == B.ERR_ARG
    assert lib.a2sgd_encode(h, g.data_ptr(), s, e.data_ptr(), s, hp, None, None, None) == B.ERR_ARG
    assert lib.a2sgd_decode_update(h, w.data_ptr(), 0, g.data_ptr(), s, e.data_ptr(), s, lm.data_ptr(), hp, 0.1, None) == B.ERR_ARG
    vp = ctypes.c_void_p
    numel = (ctypes.c_uint64 * 1)(n)
    g_tab = (vp * 2)(g[0].data_ptr(), hp)                     # worker 1's gradient tensor lives on the host
    e_tab = (vp * 2)(e[0].data_ptr(), e[1].data_ptr())
    w_tab = (vp * 1)(w.data_ptr())
    out = vp()
    assert lib.a2sgd_segments_create(h, 1, numel, g_tab, e_tab, w_tab, 0, ctypes.byref(out)) == B.ERR_ARG and not out
    B.a2sgd_step_momentum(ctx, w, m, g, e, 0.1, 0.9, 0.0)     # device buffers pass
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    ctx.destroy()
