"""Seeded synthetic inputs for the A2SGD gradient path.

This module holds no arithmetic of the method itself: it only lays out flat
parameter vectors with the tensor structure of the benchmark configurations
and fills gradient / weight buffers with seeded random values.  Both the CUDA
path and the CPU oracle are fed the *same bytes* produced here (generated once
on whichever device the caller's buffer lives on, then copied), never two
independent regenerations.

The paper trains on MNIST / CIFAR10 / PTB and observes gradients that are
"normal around zero" (Section 3, Fig. 1); those datasets are not needed for
the per-worker gradient path, so seeded synthetic values with the same shapes
stand in for them.

Every draw is keyed by (config seed, step, worker); the per-tensor scales are
drawn once per config and shared by all workers and steps.
"""
from __future__ import annotations

import dataclasses
from typing import List, Tuple

import numpy as np
import torch

BASE_SEED = 20060740


@dataclasses.dataclass(frozen=True)
class Segment:
    name: str
    numel: int
    kind: str = "weight"  # "weight" | "bn_bias" (only the kind the value recipe needs)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # position in the benchmark's config list
    P: int                     # simulated workers
    steps: int                 # steps of the parity run
    lr: float
    dist: str                  # "normal" | "laplace"
    scale_log10: Tuple[float, float]   # per-segment scale = 10**U(lo, hi)
    segments: Tuple[Segment, ...]
    zero_prob_bn_bias: float = 0.0     # exact +0.0 with this probability in bn_bias segments
    outlier_prob: float = 0.0          # each element x100 with this probability
    outlier_gain: float = 100.0
    w_std: float = 0.02

    @property
    def n(self) -> int:
        return sum(s.numel for s in self.segments)

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


def _lstm_ptb_segments() -> List[Segment]:
    # 2-layer LSTM, hidden 1500, vocab 10000: 66,034,000 parameters (the paper's Table 1 size).
    h, v = 1500, 10000
    segs = [Segment("encoder.weight", v * h)]
    for layer in range(2):
        segs += [Segment(f"rnn.weight_ih_l{layer}", 4 * h * h),
                 Segment(f"rnn.weight_hh_l{layer}", 4 * h * h),
                 Segment(f"rnn.bias_ih_l{layer}", 4 * h),
                 Segment(f"rnn.bias_hh_l{layer}", 4 * h)]
    segs += [Segment("decoder.weight", v * h), Segment("decoder.bias", v)]
    return segs


def _resnet50_segments() -> List[Segment]:
    # 53 convolutions, a BatchNorm (weight, bias) after each, fc 2048 -> 1000: 161 tensors.
    segs: List[Segment] = []

    def conv_bn(name, cin, cout, k):
        segs.append(Segment(f"{name}.conv", cout * cin * k * k))
        segs.append(Segment(f"{name}.bn.weight", cout))
        segs.append(Segment(f"{name}.bn.bias", cout, "bn_bias"))

    conv_bn("stem", 3, 64, 7)
    cin = 64
    for stage, (blocks, width) in enumerate(zip([3, 4, 6, 3], [64, 128, 256, 512])):
        for b in range(blocks):
            pre = f"layer{stage + 1}.{b}"
            conv_bn(pre + ".a", cin, width, 1)
            conv_bn(pre + ".b", width, width, 3)
            conv_bn(pre + ".c", width, 4 * width, 1)
            if b == 0:
                conv_bn(pre + ".downsample", cin, 4 * width, 1)
            cin = 4 * width
    segs += [Segment("fc.weight", 1000 * 2048), Segment("fc.bias", 1000)]
    return segs


def _vgg16_segments() -> List[Segment]:
    # 13 3x3 convolutions with biases, fc 25088 -> 4096 -> 4096 -> 1000: 32 tensors.
    segs: List[Segment] = []
    cin = 3
    for i, cout in enumerate([64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512]):
        segs += [Segment(f"conv{i}.weight", cout * cin * 9), Segment(f"conv{i}.bias", cout)]
        cin = cout
    for i, (a, b) in enumerate([(25088, 4096), (4096, 4096), (4096, 1000)]):
        segs += [Segment(f"fc{i}.weight", a * b), Segment(f"fc{i}.bias", b)]
    return segs


def _gpt2_xl_segments() -> List[Segment]:
    # 48 layers, d = 1600, vocab 50257, 1024 positions: 580 tensors, 1,557,611,200 parameters.
    d, layers, vocab, ctx = 1600, 48, 50257, 1024
    segs = [Segment("wte", vocab * d), Segment("wpe", ctx * d)]
    for l in range(layers):
        pre = f"h{l}"
        segs += [Segment(pre + ".ln_1.weight", d), Segment(pre + ".ln_1.bias", d),
                 Segment(pre + ".attn.c_attn.weight", d * 3 * d), Segment(pre + ".attn.c_attn.bias", 3 * d),
                 Segment(pre + ".attn.c_proj.weight", d * d), Segment(pre + ".attn.c_proj.bias", d),
                 Segment(pre + ".ln_2.weight", d), Segment(pre + ".ln_2.bias", d),
                 Segment(pre + ".mlp.c_fc.weight", d * 4 * d), Segment(pre + ".mlp.c_fc.bias", 4 * d),
                 Segment(pre + ".mlp.c_proj.weight", 4 * d * d), Segment(pre + ".mlp.c_proj.bias", d)]
    segs += [Segment("ln_f.weight", d), Segment("ln_f.bias", d)]
    return segs


def _build_table():
    return {
        "c1_flat_1m": Workload("c1_flat_1m", 0, P=1, steps=3, lr=0.1, dist="normal",
                               scale_log10=(-3.0, -3.0),
                               segments=(Segment("flat", 1 << 20),)),
        "c2_lstm_ptb": Workload("c2_lstm_ptb", 1, P=4, steps=10, lr=0.1, dist="normal",
                                scale_log10=(-5.0, -2.0),
                                segments=tuple(_lstm_ptb_segments())),
        "c3_resnet50": Workload("c3_resnet50", 2, P=8, steps=10, lr=0.1, dist="laplace",
                                scale_log10=(-4.0, -2.0),
                                segments=tuple(_resnet50_segments()),
                                zero_prob_bn_bias=0.3),
        "c4_vgg16": Workload("c4_vgg16", 3, P=4, steps=10, lr=0.1, dist="normal",
                             scale_log10=(-5.0, -2.0),
                             segments=tuple(_vgg16_segments()),
                             outlier_prob=1e-3),
        "c5_gpt2_xl": Workload("c5_gpt2_xl", 4, P=4, steps=5, lr=0.1, dist="normal",
                               scale_log10=(-5.0, -3.0),
                               segments=tuple(_gpt2_xl_segments())),
    }


WORKLOADS = _build_table()


def get_workload(name: str) -> Workload:
    return WORKLOADS[name]


def scaled(wl: Workload, divisor: int) -> Workload:
    """Same tensor structure with every segment length divided by ``divisor``
    (at least 1 element each).  Used for parity cases the oracle finishes in
    seconds and for profiler captures."""
    segs = tuple(dataclasses.replace(s, numel=max(1, s.numel // divisor)) for s in wl.segments)
    return dataclasses.replace(wl, name=f"{wl.name}/div{divisor}", segments=segs)


def segment_scales(wl: Workload) -> np.ndarray:
    """One scale per segment, log-uniform over ``scale_log10``, drawn once per config."""
    rng = np.random.default_rng(wl.seed)
    lo, hi = wl.scale_log10
    return (10.0 ** rng.uniform(lo, hi, size=len(wl.segments))).astype(np.float64)


def _generator(device: torch.device, *key: int) -> torch.Generator:
    gen = torch.Generator(device=device)
    seed = 0
    for k in key:  # simple injective-enough mixing of small non-negative integers
        seed = (seed * 1000003 + int(k) + 1) % (2 ** 63 - 1)
    gen.manual_seed(seed)
    return gen


def fill_gradients(wl: Workload, step: int, out: torch.Tensor) -> None:
    """Fill ``out[p, :n]`` (float32, any device) with worker p's gradient of ``step``."""
    assert out.dtype == torch.float32 and out.dim() == 2 and out.shape[0] == wl.P
    assert out.shape[1] >= wl.n
    scales = segment_scales(wl)
    for p in range(wl.P):
        gen = _generator(out.device, wl.seed, step, p)
        off = 0
        for seg, s in zip(wl.segments, scales):
            x = out[p, off:off + seg.numel]
            if wl.dist == "normal":
                x.normal_(0.0, float(s), generator=gen)
            elif wl.dist == "laplace":
                # Laplace(0, b) = b * Exp(1) with a random sign
                x.exponential_(1.0, generator=gen)
                sign = torch.empty_like(x).uniform_(-1.0, 1.0, generator=gen).sign_()
                x.mul_(sign).mul_(float(s))
            else:
                raise ValueError(wl.dist)
            if wl.outlier_prob > 0.0:
                hit = torch.empty_like(x).uniform_(0.0, 1.0, generator=gen) < wl.outlier_prob
                x[hit] *= wl.outlier_gain
            if seg.kind == "bn_bias" and wl.zero_prob_bn_bias > 0.0:
                hit = torch.empty_like(x).uniform_(0.0, 1.0, generator=gen) < wl.zero_prob_bn_bias
                x[hit] = 0.0
            off += seg.numel


def init_weights(wl: Workload, out: torch.Tensor) -> None:
    """Fill ``out[..., :n]`` with N(0, w_std) initial weights (seeded)."""
    gen = _generator(out.device, wl.seed, 10 ** 6)
    out.normal_(0.0, wl.w_std, generator=gen)


def describe(wl: Workload) -> dict:
    return {"workload": wl.name, "n": wl.n, "P": wl.P, "tensors": len(wl.segments),
            "dist": wl.dist, "lr": wl.lr}
