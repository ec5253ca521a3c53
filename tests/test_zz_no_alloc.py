"""The allocation-free encode entry point against the regular one.

Some users of this library cannot let it call cudaMalloc: their framework's caching allocator
already owns the whole GPU, or they run under a "no allocation after start-up" rule, or they
cannot afford the device synchronisation an allocation implies.  a2sgd_encode_noalloc serves
them with a fixed scratch array that lives inside the library image.  This test calls it through
the C ABI twice in a row (the second call reuses whatever the first left in the shared scratch)
and compares with a2sgd_encode, which uses a context's allocated scratch.  It is collected last
so that a run that stops at the first failure has already run every other test, and it does not
depend on any of them having run."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_07405_b200 import binding as B
from parity_util import assert_means

pytestmark = pytest.mark.gpu


def _inputs(seed, P, n, stride):
    gen = torch.Generator("cuda").manual_seed(seed)
    g = torch.empty((P, stride), device="cuda")[:, :n]
    e = torch.empty((P, stride), device="cuda")[:, :n]
    g.normal_(0.0, 1e-3, generator=gen)
    e.normal_(0.0, 3e-4, generator=gen)
    return g, e


@pytest.mark.parametrize("mode", [B.MODE_EF, B.MODE_ALG1])
@pytest.mark.parametrize("P,n,stride", [(4, 1_000_003, 1_000_032), (3, 70_001, 70_001), (1, 5, 5), (64, 4096, 4096)])
def test_noalloc_encode_matches_regular_encode_twice(mode, P, n, stride):
    ctx = B.a2sgd_create(n, P, 0, mode)
    for call in range(2):                       # second call: different data, same shared scratch
        g, e = _inputs(100 * call + P, P, n, stride)
        err = e if mode == B.MODE_EF else None
        lm_ref = torch.zeros((P, 2), device="cuda")
        cnt_ref = torch.zeros(P, dtype=torch.int64, device="cuda")
        B.a2sgd_encode(ctx, g, err, lm_ref, cnt_ref)
        lm_buf = torch.full((P + 2, 2), float("nan"), device="cuda")
        cnt = torch.full((P,), -1, dtype=torch.int64, device="cuda")
        B.a2sgd_encode_noalloc(g, err, lm_buf[1:P + 1], cnt, mode=mode)
        torch.cuda.synchronize()
        assert torch.equal(cnt, cnt_ref)                                   # integers: equal
        assert_means(lm_buf[1:P + 1].cpu().numpy(), lm_ref.cpu().numpy())   # 1e-6, as everywhere
        assert torch.isnan(lm_buf[0]).all() and torch.isnan(lm_buf[P + 1]).all()
        # and directly against the CPU oracle on the same inputs
        lm_o, cnt_o, _ = oracle.encode(g.cpu().numpy(), e.cpu().numpy() if mode == B.MODE_EF else None, mode=mode)
        assert np.array_equal(cnt.cpu().numpy().astype(np.uint64), cnt_o)
        assert_means(lm_buf[1:P + 1].cpu().numpy(), lm_o)
    ctx.destroy()


def test_noalloc_calls_leave_device_memory_as_it_was():
    """What the entry point exists for: after a first call has done its one-time set-up, further
    calls neither take nor return device memory — seen from the driver (free bytes) and from the
    caller's own allocator."""
    P, n = 4, 1 << 20
    g, e = _inputs(7, P, n, n)
    lm = torch.zeros((P, 2), device="cuda")
    cnt = torch.zeros(P, dtype=torch.int64, device="cuda")
    B.a2sgd_encode_noalloc(g, e, lm, cnt)          # first call on this device: symbol look-up, module load
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    held_before = torch.cuda.memory_allocated()
    for _ in range(2):
        B.a2sgd_encode_noalloc(g, e, lm, cnt)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert torch.cuda.memory_allocated() == held_before


def test_noalloc_rejects_what_the_fixed_scratch_cannot_hold():
    P = B.NOALLOC_MAX_P + 1
    g = torch.zeros((P, 64), device="cuda")
    lm = torch.zeros((P, 2), device="cuda")
    with pytest.raises(B.A2SGDError) as ei:
        B.a2sgd_encode_noalloc(g, g, lm)
    assert ei.value.status == B.ERR_TOO_LARGE
    with pytest.raises(B.A2SGDError) as ei:                 # EF mode needs the error buffer
        B.a2sgd_encode_noalloc(g[:2], None, lm[:2])
    assert ei.value.status == B.ERR_ARG
