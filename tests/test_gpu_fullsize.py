"""Parity at the benchmark's full sizes, in the launch configuration bench.py times
(EF mode, one shared w, rows 128-byte aligned): the two local and two global means and the
positive counts against a full oracle pass over all n*P elements; updated w and err against the
oracle on sampled windows (first and last elements, the region around the CTA-stride seams, and
random indices), which the oracle computes element by element from the same inputs."""
import numpy as np
import psutil
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from paper_2006_07405_b200 import workloads as W
from parity_util import assert_means, assert_state

pytestmark = pytest.mark.gpu


def _sample_indices(n, launch, seed):
    rng = np.random.default_rng(seed)
    win = 4096
    parts = [np.arange(0, min(win, n)), np.arange(max(0, n - win), n)]
    # seams of the persistent grids: multiples of (CTAs * 256 threads * 8 elements)
    for ctas in {launch["encode_ctas"], launch["decode_ctas"]}:
        seam = ctas * launch["threads"] * 8
        for k in (1, 2, max(1, n // seam)):
            lo = k * seam - 512
            if 0 <= lo and lo + 1024 <= n:
                parts.append(np.arange(lo, lo + 1024))
    parts.append(rng.integers(0, n, size=200_000))
    return np.unique(np.concatenate(parts))


@pytest.mark.parametrize("name", ["c2_lstm_ptb", "c3_resnet50", "c4_vgg16", "c5_gpt2_xl"])
def test_full_size_step_matches_oracle(name):
    wl = W.get_workload(name)
    n, P = wl.n, wl.P
    need_dev = (2 * P + 1) * n * 4 * 1.1 + (2 << 30)
    free_dev, _ = torch.cuda.mem_get_info()
    if need_dev > free_dev:
        pytest.skip(f"needs {need_dev / 1e9:.0f} GB of device memory")
    if psutil.virtual_memory().available < 3 * n * 4 + (8 << 30):
        pytest.skip("not enough host memory for one worker's vectors")
    dev = torch.device("cuda:0")
    g = B.padded_rows(P, n, dev)
    e = B.padded_rows(P, n, dev)
    w = torch.empty(n, device=dev)
    W.fill_gradients(wl, 0, g)
    W.init_weights(wl, w)
    # a seeded, non-trivial retained error: a third of the gradient scale, element by element
    gen = torch.Generator(device=dev).manual_seed(wl.seed + 99)
    for p in range(P):
        e[p].normal_(0.0, 1.0, generator=gen)
        e[p].mul_(g[p].abs()).mul_(0.3)

    ctx = B.a2sgd_create(n, P, 0, B.MODE_EF)
    launch = B.a2sgd_launch_info(ctx, shared_w=True)
    assert not launch["single_launch"]
    idx = _sample_indices(n, launch, wl.seed)
    idx_dev = torch.from_numpy(idx).to(dev)
    g_s = g[:, idx_dev].cpu().numpy()
    e_s = e[:, idx_dev].cpu().numpy()
    w_s = w[idx_dev].cpu().numpy()

    # full oracle pass for the means, one worker at a time (bounded host memory)
    lm_ref = np.zeros((P, 2), np.float32)
    cnt_ref = np.zeros(P, np.uint64)
    for p in range(P):
        gh = g[p:p + 1].cpu().numpy()
        eh = e[p:p + 1].cpu().numpy()
        lm_p, cnt_p, _ = oracle.encode(gh, eh, mode=oracle.MODE_EF)
        lm_ref[p], cnt_ref[p] = lm_p[0], cnt_p[0]
        del gh, eh
    gm_ref = oracle.global_average(lm_ref)

    B.a2sgd_step(ctx, w, g, e, wl.lr)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK
    assert np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref, f"{name} local means")
    assert_means(gm, gm_ref, f"{name} global means")

    # sampled outputs: the oracle's decode on exactly those elements, with its own full-pass means
    oracle.decode_update(w_s, g_s, e_s, lm_ref, gm_ref, wl.lr, mode=oracle.MODE_EF)
    assert_state(w[idx_dev].cpu().numpy(), w_s, e[:, idx_dev].cpu().numpy(), e_s, gm_ref, f"{name} sampled")

    # properties that hold at any size, on the whole output (computed with torch reductions only
    # as plumbing): the residual of worker p sums to n+ (mu+ - m+) over its positive group
    for p in range(P):
        v_pos_sum = float(lm_ref[p, 0]) * int(cnt_ref[p])
        got = float(e[p].double().sum().item())
        expect = (float(lm_ref[p, 0]) - float(gm_ref[0])) * int(cnt_ref[p]) \
            - (float(lm_ref[p, 1]) - float(gm_ref[1])) * (n - int(cnt_ref[p]))
        scale = max(v_pos_sum, 1e-30)
        assert abs(got - expect) <= 2e-5 * scale, (name, p, got, expect)
    ctx.destroy()


@pytest.mark.parametrize("mode,replicated", [(B.MODE_ALG1, False), (B.MODE_EF, True), (B.MODE_ALG1, True)])
def test_full_size_other_modes_and_layouts(mode, replicated):
    """c2 at full size in the configurations the benchmark does not time: the paper-literal
    Algorithm 1 mode and one weight replica per worker.  Same protocol: full oracle pass for the
    means, sampled windows for w and err."""
    wl = W.get_workload("c2_lstm_ptb")
    n, P = wl.n, wl.P
    dev = torch.device("cuda:0")
    g = B.padded_rows(P, n, dev)
    e = B.padded_rows(P, n, dev)
    W.fill_gradients(wl, 1, g)
    gen = torch.Generator(device=dev).manual_seed(wl.seed + 7)
    e.normal_(0.0, 1e-4, generator=gen)
    if replicated:
        w = B.padded_rows(P, n, dev)
        w.normal_(0.0, wl.w_std, generator=gen)
    else:
        w = torch.empty(n, device=dev)
        W.init_weights(wl, w)
    ctx = B.a2sgd_create(n, P, 0, mode)
    launch = B.a2sgd_launch_info(ctx, shared_w=not replicated)
    idx = _sample_indices(n, launch, wl.seed + 1)
    idx_dev = torch.from_numpy(idx).to(dev)
    g_s = g[:, idx_dev].cpu().numpy()
    e_s = e[:, idx_dev].cpu().numpy()
    w_s = (w[:, idx_dev] if replicated else w[idx_dev]).cpu().numpy()
    gh = g.cpu().numpy()
    eh = e.cpu().numpy() if mode == B.MODE_EF else None
    lm_ref, cnt_ref, _ = oracle.encode(gh, eh, mode=mode)
    gm_ref = oracle.global_average(lm_ref)
    del gh, eh
    B.a2sgd_step(ctx, w, g, e, wl.lr)
    lm, gm, cnt, status = B.a2sgd_read_stats(ctx)
    assert status == B.OK and np.array_equal(cnt, cnt_ref)
    assert_means(lm, lm_ref)
    assert_means(gm, gm_ref)
    oracle.decode_update(w_s, g_s, e_s, lm_ref, gm_ref, wl.lr, mode=mode)
    w_got = (w[:, idx_dev] if replicated else w[idx_dev]).cpu().numpy()
    assert_state(w_got, w_s, e[:, idx_dev].cpu().numpy(), e_s, gm_ref, f"mode {mode} replicated {replicated}")
    ctx.destroy()
