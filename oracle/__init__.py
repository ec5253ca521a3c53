"""ctypes front end of the A2SGD CPU oracle — TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do, and this
package imports nothing of theirs.  All arithmetic lives in
``a2sgd_oracle.c`` (plain C, fp64 accumulation, the paper's Section 3.1,
Eq. 2 and Algorithm 1 written out); this file only compiles it with gcc and
marshals numpy arrays.

Arrays: ``grad`` and ``err`` are float32 ``[P, n]`` (row p = worker p; the
row stride may exceed n); ``w`` is float32 ``[n]`` (one shared weight
vector) or ``[P, n]`` (one replica per worker).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

MODE_EF = 0
MODE_ALG1 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "a2sgd_oracle.c")
_LIB = os.path.join(_HERE, "liba2sgd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off",
             "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f32p = ctypes.POINTER(ctypes.c_float)
        u64p = ctypes.POINTER(ctypes.c_uint64)
        u32p = ctypes.POINTER(ctypes.c_uint32)
        lib.a2sgd_oracle_encode.restype = ctypes.c_int
        lib.a2sgd_oracle_encode.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint32, f32p, ctypes.c_int64,
            f32p, ctypes.c_int64, f32p, u64p, u32p]
        lib.a2sgd_oracle_global_average.restype = ctypes.c_int
        lib.a2sgd_oracle_global_average.argtypes = [ctypes.c_uint32, f32p, f32p]
        lib.a2sgd_oracle_decode_update.restype = ctypes.c_int
        lib.a2sgd_oracle_decode_update.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint32, f32p, ctypes.c_int64,
            f32p, ctypes.c_int64, f32p, ctypes.c_int64, f32p, f32p, ctypes.c_float]
        lib.a2sgd_oracle_step.restype = ctypes.c_int
        lib.a2sgd_oracle_step.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint32, f32p, ctypes.c_int64,
            f32p, ctypes.c_int64, f32p, ctypes.c_int64, ctypes.c_float,
            f32p, f32p, u64p]
        lib.a2sgd_oracle_decode_update_momentum.restype = ctypes.c_int
        lib.a2sgd_oracle_decode_update_momentum.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint32, f32p, ctypes.c_int64, f32p, ctypes.c_int64,
            f32p, ctypes.c_int64, f32p, ctypes.c_int64, f32p, f32p, ctypes.c_float, ctypes.c_float, ctypes.c_float]
        lib.a2sgd_oracle_dense_sync.restype = ctypes.c_int
        lib.a2sgd_oracle_dense_sync.argtypes = [
            ctypes.c_uint64, ctypes.c_uint32, f32p, ctypes.c_int64, f32p, ctypes.c_int64, ctypes.c_float]
        _lib = lib
    return _lib


_SRC_OMP = os.path.join(_HERE, "a2sgd_oracle_omp.c")
_LIB_OMP = os.path.join(_HERE, "liba2sgd_oracle_omp.so")
_lib_omp = None


def build_omp(force: bool = False) -> str:
    """Compile the OpenMP timing copy of the step (separate library; the pinned oracle is untouched)."""
    if force or not os.path.exists(_LIB_OMP) or os.path.getmtime(_LIB_OMP) < os.path.getmtime(_SRC_OMP):
        tmp = f"{_LIB_OMP}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
             "-shared", "-fPIC", "-o", tmp, _SRC_OMP])
        os.replace(tmp, _LIB_OMP)
    return _LIB_OMP


def _load_omp():
    global _lib_omp
    if _lib_omp is None:
        lib = ctypes.CDLL(build_omp())
        f32p = ctypes.POINTER(ctypes.c_float)
        lib.a2sgd_oracle_omp_threads.restype = ctypes.c_int
        lib.a2sgd_oracle_omp_step.restype = ctypes.c_int
        lib.a2sgd_oracle_omp_step.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint32, f32p, ctypes.c_int64,
            f32p, ctypes.c_int64, f32p, ctypes.c_int64, ctypes.c_float,
            f32p, f32p, ctypes.POINTER(ctypes.c_uint64)]
        _lib_omp = lib
    return _lib_omp


def omp_threads() -> int:
    """Threads the OpenMP copy will use."""
    return int(_load_omp().a2sgd_oracle_omp_threads())


def step_all_cores(w, grad, err, lr, *, mode=MODE_EF, n=None):
    """The OpenMP timing copy of ``step`` (all host cores).  Same interface and, up to the order of
    the fp64 additions inside the group sums, the same results."""
    lib = _load_omp()
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err") if err is not None else (None, 0)
    wp, ws = _weights(w, P)
    means = np.zeros((P, 2), np.float32)
    gmeans = np.zeros(2, np.float32)
    counts = np.zeros(P, np.uint64)
    _check(lib.a2sgd_oracle_omp_step(
        mode, n, P, wp, ws, gp, gs, ep, es, lr,
        means.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        gmeans.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        counts.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))), "omp step")
    return means, gmeans, counts


def _rows(a: np.ndarray, name: str):
    """float32 [P, n] with unit inner stride -> (pointer, row stride in elements)."""
    if a.dtype != np.float32 or a.ndim != 2 or a.strides[1] != 4 or a.strides[0] % 4:
        raise ValueError(f"{name}: need float32 [P, n] with contiguous rows")
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), a.strides[0] // 4


def _weights(w: np.ndarray, P: int):
    if w.dtype != np.float32 or w.strides[-1] != 4:
        raise ValueError("w: need float32 with contiguous rows")
    ptr = w.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    if w.ndim == 1:
        return ptr, 0
    if w.ndim == 2 and w.shape[0] == P:
        return ptr, w.strides[0] // 4
    raise ValueError("w: need [n] (shared) or [P, n] (replicated)")


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with status {rc}")


def encode(grad, err=None, *, mode=MODE_EF, n=None, want_mask=False):
    """Local means, positive counts and (optionally) the packed pos mask."""
    lib = _load()
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err") if err is not None else (None, 0)
    means = np.zeros((P, 2), np.float32)
    counts = np.zeros(P, np.uint64)
    mask = np.zeros((P, (n + 31) // 32), np.uint32) if want_mask else None
    _check(lib.a2sgd_oracle_encode(
        mode, n, P, gp, gs, ep, es,
        means.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        counts.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)),
        mask.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)) if want_mask else None),
        "encode")
    return means, counts, mask


def global_average(local_means):
    lib = _load()
    lm = np.ascontiguousarray(local_means, np.float32)
    out = np.zeros(2, np.float32)
    _check(lib.a2sgd_oracle_global_average(
        lm.shape[0], lm.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        out.ctypes.data_as(ctypes.POINTER(ctypes.c_float))), "global_average")
    return out


def decode_update(w, grad, err, local_means, global_means, lr, *, mode=MODE_EF, n=None):
    """In place: w (and err, when given) are updated."""
    lib = _load()
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err") if err is not None else (None, 0)
    wp, ws = _weights(w, P)
    lm = np.ascontiguousarray(local_means, np.float32) if local_means is not None else None
    gm = np.ascontiguousarray(global_means, np.float32)
    _check(lib.a2sgd_oracle_decode_update(
        mode, n, P, wp, ws, gp, gs, ep, es,
        lm.ctypes.data_as(ctypes.POINTER(ctypes.c_float)) if lm is not None else None,
        gm.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), lr), "decode_update")


def decode_update_momentum(w, mom, grad, err, local_means, global_means, lr, beta, weight_decay, *,
                           mode=MODE_EF, n=None):
    """Decode / residual / update with heavy-ball momentum and weight decay, in place:
    m <- beta*m + g_hat + weight_decay*w;  w <- w - lr*m.  ``mom`` has the layout of ``w``."""
    lib = _load()
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err") if err is not None else (None, 0)
    wp, ws = _weights(w, P)
    mp, ms = _weights(mom, P)
    lm = np.ascontiguousarray(local_means, np.float32) if local_means is not None else None
    gm = np.ascontiguousarray(global_means, np.float32)
    _check(lib.a2sgd_oracle_decode_update_momentum(
        mode, n, P, wp, ws, mp, ms, gp, gs, ep, es,
        lm.ctypes.data_as(ctypes.POINTER(ctypes.c_float)) if lm is not None else None,
        gm.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), lr, beta, weight_decay), "decode_update_momentum")


def step_momentum(w, mom, grad, err, lr, beta, weight_decay, *, mode=MODE_EF, n=None):
    """encode -> global_average -> decode_update_momentum, the three oracle calls in order.
    Returns (local_means, global_means, pos_counts)."""
    lm, cnt, _ = encode(grad, err if mode == MODE_EF else None, mode=mode, n=n)
    gm = global_average(lm)
    decode_update_momentum(w, mom, grad, err, lm, gm, lr, beta, weight_decay, mode=mode, n=n)
    return lm, gm, cnt


def step(w, grad, err, lr, *, mode=MODE_EF, n=None):
    """One loop body of Algorithm 1 for all P workers, in place.

    Returns (local_means [P,2], global_means [2], pos_counts [P])."""
    lib = _load()
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    gp, gs = _rows(grad, "grad")
    ep, es = _rows(err, "err") if err is not None else (None, 0)
    wp, ws = _weights(w, P)
    means = np.zeros((P, 2), np.float32)
    gmeans = np.zeros(2, np.float32)
    counts = np.zeros(P, np.uint64)
    _check(lib.a2sgd_oracle_step(
        mode, n, P, wp, ws, gp, gs, ep, es, lr,
        means.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        gmeans.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        counts.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))), "step")
    return means, gmeans, counts


def dense_sync(w, grad, lr, *, n=None):
    """Algorithm 1 lines 9-10: w <- w - lr * mean over workers of grad, in place."""
    lib = _load()
    P = grad.shape[0]
    n = grad.shape[1] if n is None else n
    gp, gs = _rows(grad, "grad")
    wp, ws = _weights(w, P)
    _check(lib.a2sgd_oracle_dense_sync(n, P, wp, ws, gp, gs, lr), "dense_sync")
