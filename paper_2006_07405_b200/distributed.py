"""A2SGD with real workers: one process (one GPU) per worker, as in Algorithm 1 of the paper.

Every rank keeps its own gradient, error vector and model replica; the only thing that crosses
between ranks per iteration is the pair of local means — 64 bits per worker (Algorithm 1 line 5).
The compute runs in the same CUDA kernels as the single-GPU path (encode, global average,
decode/update through the C ABI); this module only adds the exchange, with torch.distributed as
the transport:

* ``exchange="allgather"`` (default): every rank gathers all 2W scalars and averages them itself
  with the library's fixed-order fp64 kernel, so all ranks hold bit-identical global means.  The
  paper names all-gather as the alternative it expects to be faster than its all-reduce.
* ``exchange="allreduce"``: the paper's own choice, Allreduce(average) of the two means: the
  collective sums the pairs (widened to fp64, so its summation order cannot show at fp32
  precision) and the library divides by the worker count and rounds once.

With the NCCL backend the two scalars never leave the device.  With gloo (used by the tests) they
take a round trip through host memory.

The benchmarked configuration of this repository simulates the P workers on ONE GPU and needs none
of this; ``bench.py --gpus N`` (N > 1) additionally times both exchanges with one worker per GPU.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import binding as B


def exchange_local_means(local_means: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of each rank's [P_local, 2] local means -> [world * P_local, 2], in rank order."""
    world = dist.get_world_size(group)
    on_device = local_means.is_cuda and dist.get_backend(group) == "nccl"
    src = local_means.contiguous() if on_device else local_means.detach().cpu().contiguous()
    out = torch.empty((world * src.shape[0], 2), dtype=src.dtype, device=src.device)
    dist.all_gather_into_tensor(out, src, group=group)
    return out if on_device else out.to(local_means.device)


def sum_local_means(local_means: torch.Tensor, group=None) -> torch.Tensor:
    """All-reduce (SUM) of the [1, 2] local means widened to float64 -> [2] float64 sums over the
    ranks.  Only the transport happens here; the division that turns the sum into the paper's
    Allreduce(average) is done by the library (a2sgd_global_average_from_sums)."""
    on_device = local_means.is_cuda and dist.get_backend(group) == "nccl"
    buf = local_means.reshape(-1).to(torch.float64) if on_device else local_means.detach().cpu().reshape(-1).to(torch.float64)
    dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
    return buf if on_device else buf.to(local_means.device)


class DistributedA2SGD:
    """One worker per rank.  ``n`` parameters; this rank's worker is rank ``dist.get_rank()``."""

    def __init__(self, n: int, device: int = 0, mode: int = B.MODE_EF, group=None, exchange: str = "allgather"):
        if exchange not in ("allgather", "allreduce"):
            raise ValueError("exchange must be 'allgather' or 'allreduce'")
        self.group, self.exchange, self.mode = group, exchange, mode
        self.world = dist.get_world_size(group)
        self.local = B.a2sgd_create(n, 1, device, mode | B.FORCE_TWO_PASS)
        # a second, scratch-only context whose worker count is the world size: it averages the
        # gathered pairs in rank order (fp64, one rounding) exactly as the single-GPU path does
        self.avg = B.a2sgd_create(n, self.world, device, mode | B.FORCE_TWO_PASS) if exchange == "allgather" else None
        dev = torch.device("cuda", device)
        self.local_means = torch.zeros((1, 2), device=dev)
        self.global_means = torch.zeros(2, device=dev)
        self.pos_count = torch.zeros(1, dtype=torch.int64, device=dev)

    def exchange_means(self) -> None:
        """Algorithm 1 line 5: this rank's ``local_means`` -> every rank's ``global_means``."""
        if self.exchange == "allgather":
            gathered = exchange_local_means(self.local_means, self.group)
            B.a2sgd_global_average(self.avg, gathered, self.global_means)
        else:
            sums = sum_local_means(self.local_means, self.group)
            B.a2sgd_global_average_from_sums(self.local, sums, self.world, self.global_means)

    def step(self, w: torch.Tensor, grad: torch.Tensor, err: Optional[torch.Tensor], lr: float) -> None:
        """Algorithm 1 lines 3-7 at this worker.  w: [n]; grad, err: [1, n] (err None only in ALG1 mode)."""
        B.a2sgd_encode(self.local, grad, err, self.local_means, self.pos_count)
        self.exchange_means()
        B.a2sgd_decode_update(self.local, w, grad, err, self.local_means, self.global_means, lr)

    def dense_sync(self, w: torch.Tensor, grad: torch.Tensor, lr: float) -> None:
        """Algorithm 1 lines 9-10: dense all-reduce of the gradient, then the SGD step with the
        all-reduced sum divided by the worker count inside the library."""
        g = grad.reshape(-1).clone()
        if dist.get_backend(self.group) == "nccl":
            dist.all_reduce(g, op=dist.ReduceOp.SUM, group=self.group)
        else:
            h = g.cpu()
            dist.all_reduce(h, op=dist.ReduceOp.SUM, group=self.group)
            g.copy_(h)
        B.a2sgd_dense_sync_reduced(self.local, w, g, self.world, lr)

    def destroy(self) -> None:
        self.local.destroy()
        if self.avg is not None:
            self.avg.destroy()
