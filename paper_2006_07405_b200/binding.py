"""Thin ctypes binding of liba2sgd (the C ABI declared in include/a2sgd.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are used for device memory and streams, nothing else.  There
is no fallback: if the shared library has not been built, or a call returns a
negative status, an exception is raised.

Layout conventions (same as the header): ``grad`` / ``err`` are float32 CUDA
tensors ``[P, >= n]`` with unit inner stride (row p = worker p); ``w`` is
``[>= n]`` (one shared vector) or ``[P, >= n]`` (one replica per worker).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

OK = 0
ERR_ARG, ERR_ALIGN, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE, ERR_NOMEM, ERR_TOO_LARGE, ERR_BOUNDS = -1, -2, -3, -4, -5, -6, -7, -8
MODE_EF = 0
MODE_ALG1 = 1
FORCE_TWO_PASS = 1 << 4
FORCE_COOPERATIVE = 1 << 5
DEFERRED_RESIDUAL = 1 << 7
CHECK_POINTERS = 1 << 8
TEST_BARRIER_NEVER_OPENS = 1 << 9
DEBUG_CHECKS = 1 << 10
TEST_SHRINK_EXTENTS = 1 << 11
ROW_ALIGN_ELEMS = 32   # 128 bytes: rows that start on a cache-line boundary take the widest vector kernels

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liba2sgd.so")
_lib = None

_vp = ctypes.c_void_p
_i64 = ctypes.c_int64


class A2SGDError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


def lib() -> ctypes.CDLL:
    """Loads liba2sgd.so; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2006_07405_b200.build` "
                "(nvcc, sm_100a). This package has no CPU fallback.")
        l = ctypes.CDLL(LIB_PATH)
        l.a2sgd_create.restype = ctypes.c_int
        l.a2sgd_create.argtypes = [ctypes.POINTER(_vp), ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int, ctypes.c_uint32]
        l.a2sgd_destroy.restype = ctypes.c_int
        l.a2sgd_destroy.argtypes = [_vp]
        l.a2sgd_encode.restype = ctypes.c_int
        l.a2sgd_encode.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _vp, _vp, _vp]
        l.a2sgd_global_average.restype = ctypes.c_int
        l.a2sgd_global_average.argtypes = [_vp, _vp, _vp, _vp]
        l.a2sgd_decode_update.restype = ctypes.c_int
        l.a2sgd_decode_update.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _vp, ctypes.c_float, _vp]
        l.a2sgd_step.restype = ctypes.c_int
        l.a2sgd_step.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp]
        l.a2sgd_decode_update_momentum.restype = ctypes.c_int
        l.a2sgd_decode_update_momentum.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _vp,
                                                   ctypes.c_float, ctypes.c_float, ctypes.c_float, _vp]
        l.a2sgd_step_momentum.restype = ctypes.c_int
        l.a2sgd_step_momentum.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _i64,
                                          ctypes.c_float, ctypes.c_float, ctypes.c_float, _vp]
        l.a2sgd_global_average_from_sums.restype = ctypes.c_int
        l.a2sgd_global_average_from_sums.argtypes = [_vp, _vp, ctypes.c_uint32, _vp, _vp]
        l.a2sgd_dense_sync_reduced.restype = ctypes.c_int
        l.a2sgd_dense_sync_reduced.argtypes = [_vp, _vp, _vp, ctypes.c_uint32, ctypes.c_float, _vp]
        l.a2sgd_step_host.restype = ctypes.c_int
        l.a2sgd_step_host.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp, _vp]
        l.a2sgd_read_stats.restype = ctypes.c_int
        l.a2sgd_read_stats.argtypes = [_vp, _vp, _vp, _vp, ctypes.POINTER(ctypes.c_int), _vp]
        l.a2sgd_launch_info.restype = ctypes.c_int
        l.a2sgd_launch_info.argtypes = [_vp, _i64, ctypes.POINTER(ctypes.c_uint32)]
        l.a2sgd_encode_noalloc.restype = ctypes.c_int
        l.a2sgd_encode_noalloc.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, _vp, _i64, _vp, _i64,
                                           _vp, _vp, _vp]
        l.a2sgd_dense_sync.restype = ctypes.c_int
        l.a2sgd_dense_sync.argtypes = [_vp, _vp, _i64, _vp, _i64, ctypes.c_float, _vp]
        l.a2sgd_segments_create.restype = ctypes.c_int
        l.a2sgd_segments_create.argtypes = [_vp, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint64),
                                            ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                            ctypes.c_int, ctypes.POINTER(_vp)]
        l.a2sgd_segments_destroy.restype = ctypes.c_int
        l.a2sgd_segments_destroy.argtypes = [_vp]
        l.a2sgd_encode_segments.restype = ctypes.c_int
        l.a2sgd_encode_segments.argtypes = [_vp, _vp, _vp, _vp, _vp]
        l.a2sgd_decode_update_segments.restype = ctypes.c_int
        l.a2sgd_decode_update_segments.argtypes = [_vp, _vp, _vp, _vp, ctypes.c_float, _vp, _vp]
        l.a2sgd_step_segments_per_tensor.restype = ctypes.c_int
        l.a2sgd_step_segments_per_tensor.argtypes = [_vp, _vp, ctypes.c_float, _vp, _vp]
        l.a2sgd_read_segment_stats.restype = ctypes.c_int
        l.a2sgd_read_segment_stats.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp]
        l.a2sgd_step_segments.restype = ctypes.c_int
        l.a2sgd_step_segments.argtypes = [_vp, _vp, ctypes.c_float, _vp]
        for fn in (l.a2sgd_step_bf16, l.a2sgd_step_f16):
            fn.restype = ctypes.c_int
            fn.argtypes = [_vp, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp]
        l.a2sgd_materialize_err.restype = ctypes.c_int
        l.a2sgd_materialize_err.argtypes = [_vp, _vp, _i64, _vp]
        l.a2sgd_step_segments_lr.restype = ctypes.c_int
        l.a2sgd_step_segments_lr.argtypes = [_vp, _vp, _vp, _vp]
        l.a2sgd_status_string.restype = ctypes.c_char_p
        l.a2sgd_status_string.argtypes = [ctypes.c_int]
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().a2sgd_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != OK:
        raise A2SGDError(status, what)


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _rows(t: Optional[torch.Tensor], name: str) -> Tuple[Optional[int], int]:
    """float32 CUDA [P, n] with unit inner stride -> (address, worker stride in elements)."""
    if t is None:
        return None, 0
    if t.dtype != torch.float32 or not t.is_cuda or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name}: need a float32 CUDA tensor [P, n] with unit inner stride")
    return t.data_ptr(), t.stride(0)


def _weights(w: torch.Tensor) -> Tuple[int, int]:
    if w.dtype != torch.float32 or not w.is_cuda:
        raise ValueError("w: need a float32 CUDA tensor")
    if w.dim() == 1:
        return w.data_ptr(), 0
    if w.dim() == 2:
        return w.data_ptr(), w.stride(0)
    raise ValueError("w: need [n] (shared) or [P, n] (replicated)")


def padded_rows(P: int, n: int, device, fill: Optional[float] = None) -> torch.Tensor:
    """A float32 [P, n] view whose rows start 128-byte aligned (row stride = n rounded up to 32
    elements).  Device memory only; the layout the fast kernels are measured with."""
    stride = (n + ROW_ALIGN_ELEMS - 1) // ROW_ALIGN_ELEMS * ROW_ALIGN_ELEMS
    buf = torch.empty((P, stride), dtype=torch.float32, device=device)
    if fill is not None:
        buf.fill_(fill)
    return buf[:, :n]


class Context:
    """Owns an ``a2sgd_ctx``.  ``n`` elements per worker, ``P`` workers."""

    def __init__(self, n: int, P: int, device: int = 0, flags: int = MODE_EF):
        self.n, self.P, self.device, self.flags = int(n), int(P), int(device), int(flags)
        self._h = _vp()
        _check(lib().a2sgd_create(ctypes.byref(self._h), self.n, self.P, self.device, self.flags), "a2sgd_create")

    @property
    def handle(self):
        if not self._h:
            raise RuntimeError("context destroyed")
        return self._h

    def destroy(self) -> None:
        if self._h:
            lib().a2sgd_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def a2sgd_create(n: int, P: int, device: int = 0, flags: int = MODE_EF) -> Context:
    return Context(n, P, device, flags)


def a2sgd_destroy(ctx: Context) -> None:
    ctx.destroy()


def a2sgd_encode(ctx: Context, grad: torch.Tensor, err: Optional[torch.Tensor], local_means: torch.Tensor,
                 pos_counts: Optional[torch.Tensor] = None, pos_mask: Optional[torch.Tensor] = None,
                 stream=None) -> None:
    """local_means: float32 CUDA [P, 2]; pos_counts: int64 CUDA [P]; pos_mask: int32 CUDA [P, ceil(n/32)]."""
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_encode(ctx.handle, gp, gs, ep, es, local_means.data_ptr(),
                              pos_counts.data_ptr() if pos_counts is not None else None,
                              pos_mask.data_ptr() if pos_mask is not None else None, _stream(stream)),
           "a2sgd_encode")


NOALLOC_MAX_P = 64


def a2sgd_encode_noalloc(grad: torch.Tensor, err: Optional[torch.Tensor], local_means: torch.Tensor,
                         pos_counts: Optional[torch.Tensor] = None, mode: int = MODE_EF, n: Optional[int] = None,
                         stream=None) -> None:
    """Encode without a context and without any allocation inside the library (its scratch is a
    fixed array in the library image).  For callers that may not call cudaMalloc; runs on the
    current device; calls that overlap on the GPU race on the shared scratch.  Output tensors are
    the caller's: local_means float32 CUDA [P, 2], pos_counts int64 CUDA [P]."""
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err")
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    _check(lib().a2sgd_encode_noalloc(int(n), int(P), int(mode), gp, gs, ep, es, local_means.data_ptr(),
                                      pos_counts.data_ptr() if pos_counts is not None else None,
                                      _stream(stream)), "a2sgd_encode_noalloc")


def a2sgd_global_average(ctx: Context, local_means: torch.Tensor, global_means: torch.Tensor, stream=None) -> None:
    _check(lib().a2sgd_global_average(ctx.handle, local_means.data_ptr(), global_means.data_ptr(), _stream(stream)),
           "a2sgd_global_average")


def a2sgd_global_average_from_sums(ctx: Context, sums: torch.Tensor, workers: int, global_means: torch.Tensor,
                                   stream=None) -> None:
    """sums: float64 CUDA [2], the all-reduced sums of the two local means over ``workers`` workers."""
    if sums.dtype != torch.float64 or not sums.is_cuda or sums.numel() < 2:
        raise ValueError("sums: need a float64 CUDA tensor of 2 elements")
    _check(lib().a2sgd_global_average_from_sums(ctx.handle, sums.data_ptr(), int(workers), global_means.data_ptr(),
                                                _stream(stream)), "a2sgd_global_average_from_sums")


def a2sgd_dense_sync_reduced(ctx: Context, w: torch.Tensor, grad_sum: torch.Tensor, workers: int, lr: float,
                             stream=None) -> None:
    """grad_sum: float32 CUDA [n], the all-reduced sum of the workers' gradients."""
    if grad_sum.dtype != torch.float32 or not grad_sum.is_cuda or not grad_sum.is_contiguous():
        raise ValueError("grad_sum: need a contiguous float32 CUDA tensor")
    wp, _ = _weights(w)
    _check(lib().a2sgd_dense_sync_reduced(ctx.handle, wp, grad_sum.data_ptr(), int(workers), float(lr),
                                          _stream(stream)), "a2sgd_dense_sync_reduced")


def a2sgd_decode_update(ctx: Context, w: torch.Tensor, grad: torch.Tensor, err: Optional[torch.Tensor],
                        local_means: Optional[torch.Tensor], global_means: torch.Tensor, lr: float,
                        stream=None) -> None:
    wp, ws = _weights(w)
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_decode_update(ctx.handle, wp, ws, gp, gs, ep, es,
                                     local_means.data_ptr() if local_means is not None else None,
                                     global_means.data_ptr(), float(lr), _stream(stream)),
           "a2sgd_decode_update")


def a2sgd_step(ctx: Context, w: torch.Tensor, grad: torch.Tensor, err: Optional[torch.Tensor], lr: float,
               stream=None) -> None:
    wp, ws = _weights(w)
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_step(ctx.handle, wp, ws, gp, gs, ep, es, float(lr), _stream(stream)), "a2sgd_step")


def a2sgd_decode_update_momentum(ctx: Context, w: torch.Tensor, mom: torch.Tensor, grad: torch.Tensor,
                                 err: Optional[torch.Tensor], local_means: Optional[torch.Tensor],
                                 global_means: torch.Tensor, lr: float, beta: float, weight_decay: float,
                                 stream=None) -> None:
    """mom: float32 CUDA tensor with the layout of w (zero before the first step)."""
    wp, ws = _weights(w)
    mp, ms = _weights(mom)
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_decode_update_momentum(ctx.handle, wp, ws, mp, ms, gp, gs, ep, es,
                                              local_means.data_ptr() if local_means is not None else None,
                                              global_means.data_ptr(), float(lr), float(beta), float(weight_decay),
                                              _stream(stream)), "a2sgd_decode_update_momentum")


def a2sgd_step_momentum(ctx: Context, w: torch.Tensor, mom: torch.Tensor, grad: torch.Tensor,
                        err: Optional[torch.Tensor], lr: float, beta: float, weight_decay: float, stream=None) -> None:
    wp, ws = _weights(w)
    mp, ms = _weights(mom)
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_step_momentum(ctx.handle, wp, ws, mp, ms, gp, gs, ep, es, float(lr), float(beta),
                                     float(weight_decay), _stream(stream)), "a2sgd_step_momentum")


def a2sgd_step_bf16(ctx: Context, w: torch.Tensor, grad: torch.Tensor, err: Optional[torch.Tensor], lr: float,
                    stream=None) -> None:
    """a2sgd_step with bfloat16 gradients: grad is a torch.bfloat16 CUDA tensor [P, >= n]."""
    if grad.dtype != torch.bfloat16 or not grad.is_cuda or grad.dim() != 2 or (grad.shape[1] > 1 and grad.stride(1) != 1):
        raise ValueError("grad: need a bfloat16 CUDA tensor [P, n] with unit inner stride")
    wp, ws = _weights(w)
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_step_bf16(ctx.handle, wp, ws, grad.data_ptr(), grad.stride(0), ep, es, float(lr),
                                 _stream(stream)), "a2sgd_step_bf16")


def a2sgd_materialize_err(ctx: Context, err: torch.Tensor, stream=None) -> None:
    """Deferred-residual contexts: turn the buffer (holding v) back into the true residual, in place."""
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_materialize_err(ctx.handle, ep, es, _stream(stream)), "a2sgd_materialize_err")


def a2sgd_step_f16(ctx: Context, w: torch.Tensor, grad: torch.Tensor, err: Optional[torch.Tensor], lr: float,
                   stream=None) -> None:
    """a2sgd_step with half-precision gradients: grad is a torch.float16 CUDA tensor [P, >= n]."""
    if grad.dtype != torch.float16 or not grad.is_cuda or grad.dim() != 2 or (grad.shape[1] > 1 and grad.stride(1) != 1):
        raise ValueError("grad: need a float16 CUDA tensor [P, n] with unit inner stride")
    wp, ws = _weights(w)
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_step_f16(ctx.handle, wp, ws, grad.data_ptr(), grad.stride(0), ep, es, float(lr),
                                _stream(stream)), "a2sgd_step_f16")


def a2sgd_dense_sync(ctx: Context, w: torch.Tensor, grad: torch.Tensor, lr: float, stream=None) -> None:
    """Algorithm 1 lines 9-10: w <- w - lr * mean over workers of grad."""
    wp, ws = _weights(w)
    gp, gs = _rows(grad, "grad")
    _check(lib().a2sgd_dense_sync(ctx.handle, wp, ws, gp, gs, float(lr), _stream(stream)), "a2sgd_dense_sync")


class Segments:
    """Owns an ``a2sgd_segments`` plan and keeps the tensors it points at alive."""

    def __init__(self, ctx: Context, grad, err, w, w_replicated: bool):
        self.ctx = ctx
        self._keep = (grad, err, w)
        P, S = ctx.P, len(grad[0])
        numel = (ctypes.c_uint64 * S)(*[t.numel() for t in grad[0]])

        def table(rows):
            flat = [t for row in rows for t in row]
            for t in flat:
                if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
                    raise ValueError("segments: need contiguous float32 CUDA tensors")
            return (_vp * len(flat))(*[t.data_ptr() for t in flat])

        if len(grad) != P or any(len(r) != S for r in grad):
            raise ValueError("grad: need P lists of S tensors")
        g_tab = table(grad)
        e_tab = table(err) if err is not None else None
        w_tab = table(w if w_replicated else [w])
        self._h = _vp()
        _check(lib().a2sgd_segments_create(ctx.handle, S, numel, g_tab, e_tab, w_tab, 1 if w_replicated else 0,
                                           ctypes.byref(self._h)), "a2sgd_segments_create")

    @property
    def handle(self):
        if not self._h:
            raise RuntimeError("segment plan destroyed")
        return self._h

    def destroy(self) -> None:
        if self._h:
            lib().a2sgd_segments_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def a2sgd_segments_create(ctx: Context, grad, err, w, w_replicated: bool = False) -> Segments:
    """grad / err: P lists of S tensors (err None in ALG1 mode when eps is not wanted);
    w: a list of S tensors (shared) or P lists of S tensors (replicated)."""
    return Segments(ctx, grad, err, w, w_replicated)


def a2sgd_segments_destroy(plan: Segments) -> None:
    plan.destroy()


def a2sgd_step_segments(ctx: Context, plan: Segments, lr: float, stream=None) -> None:
    _check(lib().a2sgd_step_segments(ctx.handle, plan.handle, float(lr), _stream(stream)), "a2sgd_step_segments")


def a2sgd_encode_segments(ctx: Context, plan: Segments, local_means: torch.Tensor,
                          pos_counts: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().a2sgd_encode_segments(ctx.handle, plan.handle, local_means.data_ptr(),
                                       pos_counts.data_ptr() if pos_counts is not None else None, _stream(stream)),
           "a2sgd_encode_segments")


def a2sgd_decode_update_segments(ctx: Context, plan: Segments, local_means: Optional[torch.Tensor],
                                 global_means: torch.Tensor, lr: float,
                                 lr_per_segment: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().a2sgd_decode_update_segments(ctx.handle, plan.handle,
                                              local_means.data_ptr() if local_means is not None else None,
                                              global_means.data_ptr(), float(lr),
                                              lr_per_segment.data_ptr() if lr_per_segment is not None else None,
                                              _stream(stream)), "a2sgd_decode_update_segments")


def a2sgd_step_segments_per_tensor(ctx: Context, plan: Segments, lr: float,
                                   lr_per_segment: Optional[torch.Tensor] = None, stream=None) -> None:
    """Every tensor compressed on its own (its own local and global means)."""
    _check(lib().a2sgd_step_segments_per_tensor(ctx.handle, plan.handle, float(lr),
                                                lr_per_segment.data_ptr() if lr_per_segment is not None else None,
                                                _stream(stream)), "a2sgd_step_segments_per_tensor")


def a2sgd_read_segment_stats(ctx: Context, plan: Segments, S: int, stream=None):
    """Synchronises the stream.  Returns (local_means [S,P,2], global_means [S,2], pos_counts [S,P])."""
    import numpy as np
    lm = np.zeros((S, ctx.P, 2), np.float32)
    gm = np.zeros((S, 2), np.float32)
    pc = np.zeros((S, ctx.P), np.uint64)
    _check(lib().a2sgd_read_segment_stats(ctx.handle, plan.handle, lm.ctypes.data, gm.ctypes.data, pc.ctypes.data,
                                          _stream(stream)), "a2sgd_read_segment_stats")
    return lm, gm, pc


def a2sgd_step_segments_lr(ctx: Context, plan: Segments, lr_per_segment: torch.Tensor, stream=None) -> None:
    """lr_per_segment: float32 CUDA tensor of S learning rates (layer-wise policies such as LARS)."""
    if lr_per_segment.dtype != torch.float32 or not lr_per_segment.is_cuda or not lr_per_segment.is_contiguous():
        raise ValueError("lr_per_segment: need a contiguous float32 CUDA tensor")
    _check(lib().a2sgd_step_segments_lr(ctx.handle, plan.handle, lr_per_segment.data_ptr(), _stream(stream)),
           "a2sgd_step_segments_lr")


def a2sgd_step_host(ctx: Context, w: torch.Tensor, grad_host: torch.Tensor, grad_staging: torch.Tensor,
                    err: Optional[torch.Tensor], lr: float, means_host: torch.Tensor, stream=None) -> None:
    """grad_host: float32 CPU [P, >= n] (pinned for asynchronous copies); means_host: float32 CPU [2P + 2]."""
    if grad_host.is_cuda or grad_host.dtype != torch.float32 or grad_host.dim() != 2 or grad_host.stride(1) != 1:
        raise ValueError("grad_host: need a float32 CPU tensor [P, n] with unit inner stride")
    if means_host.is_cuda or means_host.dtype != torch.float32 or means_host.numel() < 2 * ctx.P + 2:
        raise ValueError("means_host: need a float32 CPU tensor of 2P + 2 elements")
    wp, ws = _weights(w)
    sp, ss = _rows(grad_staging, "grad_staging")
    ep, es = _rows(err, "err")
    _check(lib().a2sgd_step_host(ctx.handle, wp, ws, grad_host.data_ptr(), grad_host.stride(0), sp, ss, ep, es,
                                 float(lr), means_host.data_ptr(), _stream(stream)), "a2sgd_step_host")


def a2sgd_read_stats(ctx: Context, stream=None):
    """Synchronises the stream.  Returns (local_means [P,2], global_means [2], pos_counts [P], device_status)."""
    import numpy as np
    lm = np.zeros((ctx.P, 2), np.float32)
    gm = np.zeros(2, np.float32)
    pc = np.zeros(ctx.P, np.uint64)
    st = ctypes.c_int(0)
    _check(lib().a2sgd_read_stats(ctx.handle, lm.ctypes.data, gm.ctypes.data, pc.ctypes.data, ctypes.byref(st),
                                  _stream(stream)), "a2sgd_read_stats")
    return lm, gm, pc, st.value


def a2sgd_launch_info(ctx: Context, shared_w: bool = True) -> dict:
    out = (ctypes.c_uint32 * 5)()
    _check(lib().a2sgd_launch_info(ctx.handle, 0 if shared_w else ctx.n, out), "a2sgd_launch_info")
    return {"encode_ctas": out[0], "decode_ctas": out[1], "threads": out[2], "single_launch": bool(out[3]),
            "sms": out[4]}
