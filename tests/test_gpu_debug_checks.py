"""A2SGD_DEBUG_CHECKS: the checked copy of the kernels, standing in for a memory checker.

Every entry point is run on small cases with the flag on: the latched status must stay A2SGD_OK
(no kernel computes an access outside the buffers it was given) and the results must be the bits
the production kernels give.  A second test makes the check fire in a way that cannot fault: the
recorded extents are shrunk by one element per row (a test hook), so the accesses to each row's
last element are skipped and A2SGD_ERR_BOUNDS is latched, while nothing outside a buffer is ever
touched."""
import numpy as np
import pytest
import torch

from paper_2006_07405_b200 import binding as B

pytestmark = pytest.mark.gpu
EF, ALG1 = B.MODE_EF, B.MODE_ALG1


def _inputs(seed, P, n, stride, replicated):
    gen = torch.Generator("cuda").manual_seed(seed)
    mk = lambda rows, scale: torch.empty((rows, stride), device="cuda").normal_(0, scale, generator=gen)[:, :n]
    g, e = mk(P, 1e-3), mk(P, 3e-4)
    w = mk(P, 0.02) if replicated else mk(1, 0.02)[0]
    return g, e, w


CASES = [(1, 1, 1), (3, 5, 5), (4, 1027, 1027), (4, 4096, 4096 + 32), (2, 70_001, 70_004), (8, 33_333, 33_336),
         (5, 10_000, 10_001)]


@pytest.mark.parametrize("mode", [EF, ALG1])
@pytest.mark.parametrize("replicated", [False, True])
@pytest.mark.parametrize("P,n,stride", CASES)
def test_checked_kernels_stay_in_bounds_and_give_the_same_bits(mode, replicated, P, n, stride):
    outs = []
    for flags in (mode, mode | B.DEBUG_CHECKS):
        g, e, w = _inputs(n + P, P, n, stride, replicated)
        m = torch.zeros_like(w)
        ctx = B.a2sgd_create(n, P, 0, flags)
        lm = torch.zeros((P, 2), device="cuda")
        gm = torch.zeros(2, device="cuda")
        cnt = torch.zeros(P, dtype=torch.int64, device="cuda")
        mask = torch.zeros((P, (n + 31) // 32), dtype=torch.int32, device="cuda")
        B.a2sgd_step(ctx, w, g, e, 0.1)                                    # fused (single launch where it fits)
        B.a2sgd_encode(ctx, g, e if mode == EF else None, lm, cnt, mask)   # staged, with the packed mask
        B.a2sgd_global_average(ctx, lm, gm)
        B.a2sgd_decode_update(ctx, w, g, e, lm, gm, 0.1)
        B.a2sgd_step_momentum(ctx, w, m, g, e, 0.1, 0.9, 1e-4)
        B.a2sgd_dense_sync(ctx, w, g, 0.1)
        g16 = g.to(torch.bfloat16)
        B.a2sgd_step_bf16(ctx, w, g16, e, 0.1)
        *_, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK, B.status_string(status)
        outs.append([t.cpu().numpy().tobytes() for t in (w, e, m, lm, gm, cnt, mask)])
        ctx.destroy()
    assert outs[0] == outs[1]


@pytest.mark.parametrize("flag", [B.FORCE_COOPERATIVE, B.FORCE_TWO_PASS, B.DEFERRED_RESIDUAL])
def test_checked_single_launch_two_pass_and_deferred_forms(flag):
    P, n = 4, 40_000
    outs = []
    for dbg in (0, B.DEBUG_CHECKS):
        g, e, w = _inputs(5, P, n, n, False)
        ctx = B.a2sgd_create(n, P, 0, EF | flag | dbg)
        for _ in range(3):
            B.a2sgd_step(ctx, w, g, e, 0.1)
        if flag == B.DEFERRED_RESIDUAL:
            B.a2sgd_materialize_err(ctx, e)
        *_, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK, B.status_string(status)
        outs.append((w.cpu().numpy().tobytes(), e.cpu().numpy().tobytes()))
        ctx.destroy()
    assert outs[0] == outs[1]


def test_checked_segment_list_kernels():
    P, sizes = 3, [5, 2048, 70_001, 33, 4096]
    n = sum(sizes)
    outs = []
    for dbg in (0, B.DEBUG_CHECKS):
        gen = torch.Generator("cuda").manual_seed(2)
        mk = lambda scale: [torch.empty(s, device="cuda").normal_(0, scale, generator=gen) for s in sizes]
        grad, err, w = [mk(1e-3) for _ in range(P)], [mk(3e-4) for _ in range(P)], mk(0.02)
        ctx = B.a2sgd_create(n, P, 0, EF | dbg)
        plan = B.a2sgd_segments_create(ctx, grad, err, w)
        B.a2sgd_step_segments(ctx, plan, 0.1)
        B.a2sgd_step_segments_per_tensor(ctx, plan, 0.1)
        *_, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK
        outs.append(torch.cat(w + [t for row in err for t in row]).cpu().numpy().tobytes())
        plan.destroy()
        ctx.destroy()
    assert outs[0] == outs[1]


@pytest.mark.parametrize("P,n,stride", [(2, 1000, 1000), (4, 8192, 8192), (3, 70_001, 70_001)])
def test_the_check_fires_on_shrunk_extents_and_skips_the_access(P, n, stride):
    g, e, w = _inputs(9, P, n, stride, False)
    w0_last = float(w[n - 1])
    e_before = e.clone()
    ctx = B.a2sgd_create(n, P, 0, EF | B.FORCE_TWO_PASS | B.DEBUG_CHECKS | B.TEST_SHRINK_EXTENTS)
    B.a2sgd_step(ctx, w, g, e, 0.1)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.ERR_BOUNDS
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK                                    # reading clears the latch
    torch.cuda.synchronize()
    # whatever touched the last element of a row was skipped: it still holds its old value ...
    assert float(w[n - 1]) == w0_last
    # ... and elements well inside the rows were processed as usual
    assert not torch.equal(e[:, : n // 2], e_before[:, : n // 2])
    # a context without the hook runs clean on the same buffers afterwards
    ctx2 = B.a2sgd_create(n, P, 0, EF | B.DEBUG_CHECKS)
    B.a2sgd_step(ctx2, w, g, e, 0.1)
    *_, status = B.a2sgd_read_stats(ctx2)
    assert status == B.OK
    ctx.destroy()
    ctx2.destroy()


@pytest.mark.parametrize("name", ["c4_vgg16", "c5_gpt2_xl"])
def test_checked_kernels_at_full_benchmark_size(name):
    """The 64-bit index arithmetic at the largest sizes (c5: 6.2 G worker-elements, byte offsets
    beyond 2^34): the checked kernels latch nothing and produce the production kernels' bits
    (compared through exact integer checksums of the bit patterns)."""
    from paper_2006_07405_b200 import workloads as W
    wl = W.get_workload(name)
    n, P = wl.n, wl.P
    free_dev, _ = torch.cuda.mem_get_info()
    if (2 * P + 1) * n * 4 * 1.05 + (2 << 30) > free_dev:
        pytest.skip("not enough device memory")
    g = B.padded_rows(P, n, "cuda")
    e = B.padded_rows(P, n, "cuda")
    w = torch.empty(n, device="cuda")
    W.fill_gradients(wl, 0, g)

    def checksums():
        parts = [w.view(torch.int32).sum(dtype=torch.int64)] + [e[p].view(torch.int32).sum(dtype=torch.int64)
                                                              for p in range(P)]
        return [int(x.item()) for x in parts]

    sums = []
    for flags in (EF, EF | B.DEBUG_CHECKS):
        W.init_weights(wl, w)
        gen = torch.Generator(device="cuda").manual_seed(123)
        for p in range(P):
            e[p].normal_(0.0, 1e-4, generator=gen)
        ctx = B.a2sgd_create(n, P, 0, flags)
        B.a2sgd_step(ctx, w, g, e, wl.lr)
        lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
        assert status == B.OK, B.status_string(status)
        sums.append((checksums(), lm.tobytes(), gm.tobytes(), cnt.tobytes()))
        ctx.destroy()
    assert sums[0] == sums[1]


def test_checking_context_is_refused_during_stream_capture():
    """The extents of a checked call are handed to the device from a short-lived host object, so a
    captured call would replay a dangling copy: the library refuses instead."""
    P, n = 2, 4096
    g, e, w = _inputs(3, P, n, n, False)
    ctx = B.a2sgd_create(n, P, 0, EF | B.DEBUG_CHECKS)
    B.a2sgd_step(ctx, w, g, e, 0.1)                          # outside capture: fine
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            with pytest.raises(B.A2SGDError) as ei:
                B.a2sgd_step(ctx, w, g, e, 0.1, stream=side)
            w.add_(0.0)                                      # something harmless to capture
    assert ei.value.status == B.ERR_CUDA
    torch.cuda.current_stream().wait_stream(side)
    *_, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    ctx.destroy()
