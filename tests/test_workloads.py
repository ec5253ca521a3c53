"""The synthetic workloads have the stated shapes and are reproducible."""
import numpy as np
import torch

from paper_2006_07405_b200 import workloads as W


def test_sizes_and_tensor_counts():
    expect = {"c1_flat_1m": (1 << 20, 1, 1), "c2_lstm_ptb": (66_034_000, 11, 4),
              "c3_resnet50": (25_557_032, 161, 8), "c4_vgg16": (138_357_544, 32, 4),
              "c5_gpt2_xl": (1_557_611_200, 580, 4)}
    for name, (n, tensors, P) in expect.items():
        wl = W.get_workload(name)
        assert (wl.n, len(wl.segments), wl.P) == (n, tensors, P)
    r50 = W.get_workload("c3_resnet50")
    assert sum(s.numel for s in r50.segments if s.kind == "bn_bias") == 26_560
    assert sum(1 for s in r50.segments if s.name.endswith(".conv")) == 53


def test_fill_is_seeded_and_keyed_by_step_and_worker():
    wl = W.scaled(W.get_workload("c3_resnet50"), 64)
    a = torch.empty(wl.P, wl.n)
    b = torch.empty(wl.P, wl.n + 3)
    W.fill_gradients(wl, 2, a)
    W.fill_gradients(wl, 2, b)
    assert torch.equal(a, b[:, :wl.n])
    W.fill_gradients(wl, 3, b)
    assert not torch.equal(a, b[:, :wl.n])
    assert not torch.equal(a[0], a[1])
    assert torch.isfinite(a).all()
    # exact zeros appear only through the BN-bias recipe
    assert (a == 0).sum() > 0


def test_value_recipes():
    wl = W.scaled(W.get_workload("c4_vgg16"), 16)
    g = torch.empty(wl.P, wl.n)
    W.fill_gradients(wl, 0, g)
    scales = W.segment_scales(wl)
    assert scales.min() >= 1e-5 and scales.max() <= 1e-2
    off = 0
    big = int(np.argmax([s.numel for s in wl.segments]))
    for k, s in enumerate(wl.segments):
        if k == big:
            x = g[0, off:off + s.numel].double()
            frac_out = (x.abs() > 8 * scales[k]).double().mean().item()
            assert 0.5e-3 < frac_out < 2e-3          # 0.1 % outliers at 100 sigma
        off += s.numel
    w = torch.empty(wl.n)
    W.init_weights(wl, w)
    assert abs(w.std().item() - 0.02) < 1e-3
