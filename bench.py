#!/usr/bin/env python
"""Benchmark of the A2SGD per-worker gradient path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one whole pass of the hot path — encode (two local means per worker), average of
the 2P scalars, decode + residual update + SGD step — over all P simulated workers of the
workload.  Prints ONE JSON line (rank 0).

* ``value``      model parameters per second (n / step time), inputs resident in HBM.
* ``e2e``        the same metric through ``a2sgd_step_host``: every step copies that step's
                 gradients from pinned host memory and reads the 2P+2 means back.
* ``roofline``   the decode/update kernel (the larger of the two launches of a step) timed
                 alone with CUDA events: algorithmic bytes / duration against the measured
                 copy bandwidth of this machine.
* ``cpu_baseline`` the CPU oracle, as it stands, on a bounded sample of the same workload.

The default workload at N = 1 is the largest benchmark configuration, c5_gpt2_xl (1.56 G
parameters, P = 4, 56 GB resident); if the device cannot hold it the run falls back to c4_vgg16
and says so in ``config``.  The smaller configurations are timed too and reported under
``other_workloads`` with their own per-kernel roofline records.

With N > 1 (under torchrun) every rank runs an independent replica of the workload on its own
GPU — the benchmarked path has no exchange between GPUs — and the time is the max over ranks.
A second leg (``exchange_between_gpus``) then runs the method as Algorithm 1 prints it, one worker
per GPU, and times the exchange of the two local means over NCCL both ways: all-gather plus a
local fixed-order average, and all-reduce plus division.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "a2sgd_step_model_params_per_s"
UNIT = "params/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (read + write) per model element of the decode/update kernel inside one launch, from the
# ncu captures summarised under profiles/ (step_kernels_c2_lstm_ptb_div4.md for P = 4,
# step_kernels_c3_resnet50_div4.md for P = 8): reads equal the algorithmic (8P + 4) bytes; of the
# (4P + 4) bytes written about 3 (P = 4) to 7.5 (P = 8) bytes per element are still dirty in L2 when
# the kernel ends and leave during the next launch.
NCU_DECODE_TRAFFIC_PER_ELEMENT = {4: 36.00 + 16.78, 8: 68.00 + 28.49}
DEFAULT_WORKLOAD = "c5_gpt2_xl"
FALLBACK_WORKLOAD = "c4_vgg16"


def algorithmic_bytes_per_model_element(P: int, shared_w: bool = True) -> dict:
    """EF mode, fp32: K1 reads g and e of every worker; K3 reads g, e, w and writes e, w."""
    encode = 8 * P
    decode = (12 * P + 8) if shared_w else 20 * P
    return {"encode": encode, "decode": decode, "step": encode + decode}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        import torch
        self.proc = None
        self.path = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            ident = str(device_index)
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", ident, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0]))
                    smax.append(float(parts[1]))
                    power.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(smax), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- reference arm
def oracle_sample_rate(wl, target_seconds: float, gen_device="cpu", all_cores=False):
    """Times the CPU oracle (single thread, unmodified) on a prefix sample of the workload's
    flat vector: all P workers, the first n_s elements of each.  Returns a dict."""
    import numpy as np
    import torch
    import oracle
    from paper_2006_07405_b200 import workloads as W

    def run(n_s, steps=1, fn=None, skip_first=False):
        fn = fn or oracle.step
        g = torch.empty((wl.P, n_s))
        sub = W.scaled(wl, max(1, wl.n // n_s))
        gfull = torch.empty((wl.P, sub.n))
        W.fill_gradients(sub, 0, gfull)
        reps = (n_s + sub.n - 1) // sub.n
        g.copy_(gfull.repeat(1, reps)[:, :n_s])
        g = g.numpy()
        e = np.zeros_like(g)
        w = np.zeros(n_s, np.float32)
        if skip_first:
            fn(w, g, e, wl.lr, mode=oracle.MODE_EF)
            steps -= 1
        t0 = time.perf_counter()
        for _ in range(steps):
            fn(w, g, e, wl.lr, mode=oracle.MODE_EF)
        return (time.perf_counter() - t0) / steps

    probe_n = min(wl.n, 1 << 20)
    t_probe = run(probe_n)
    n_s = int(min(wl.n, max(probe_n, probe_n * target_seconds / max(t_probe, 1e-9))))
    t = run(n_s)
    out = {"value": n_s / t, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"first {n_s} of {wl.n} elements of each of the {wl.P} workers, 1 step, {t:.2f} s",
           "_n_s": n_s, "_seconds": t}
    if all_cores:
        # the same sample through the OpenMP copy of the step (a separate function: the pinned
        # oracle stays single-threaded); two steps, the second one timed
        try:
            threads = oracle.omp_threads()
            t_all = run(n_s, steps=2, fn=oracle.step_all_cores, skip_first=True)
            out["all_cores"] = {"value": n_s / t_all, "unit": UNIT, "cores": threads,
                                "kind": "OpenMP copy of the oracle's step", "seconds": t_all}
        except Exception as ex:   # no OpenMP runtime on the box: report, do not fail the bench
            out["all_cores"] = {"unavailable": str(ex)[:200]}
    return out


def run_reference(args):
    """bench.py --impl reference: the oracle on the host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2006_07405_b200 import workloads as W
    wl = W.get_workload(args.workload)
    per_step_budget = max(0.5, min(10.0, 120.0 / max(1, args.steps + args.warmup)))
    first = oracle_sample_rate(wl, per_step_budget)
    n_s = first["_n_s"]
    import numpy as np
    import torch
    import oracle
    sub = W.scaled(wl, max(1, wl.n // n_s))
    gfull = torch.empty((wl.P, sub.n))
    W.fill_gradients(sub, 0, gfull)
    g = gfull.repeat(1, (n_s + sub.n - 1) // sub.n)[:, :n_s].contiguous().numpy()
    e = np.zeros_like(g)
    w = np.zeros(n_s, np.float32)
    for _ in range(args.warmup):
        oracle.step(w, g, e, wl.lr, mode=oracle.MODE_EF)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.step(w, g, e, wl.lr, mode=oracle.MODE_EF)
    t = (time.perf_counter() - t0) / max(1, args.steps)
    value = n_s / t
    sample = f"first {n_s} of {wl.n} elements of each of the {wl.P} workers per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(W.describe(wl), note="CPU oracle, single thread, bounded sample"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- profiler helper
def run_variant(wl, variant, steps, warmup, dev):
    """--minimal --variant X: a bare loop of one entry point, for profiler captures of the kernels
    the plain step loop does not launch.  Returns ms per call."""
    import torch
    from paper_2006_07405_b200 import binding as B
    from paper_2006_07405_b200 import workloads as W
    n, P = wl.n, wl.P
    if variant == "misaligned":      # rows 4-byte aligned only, each at a different phase
        g = torch.empty((P, n + 1), device=dev)[:, :n]
        e = torch.zeros((P, n + 1), device=dev)[:, :n]
    else:
        g = B.padded_rows(P, n, dev)
        e = B.padded_rows(P, n, dev, fill=0.0)
    w = torch.empty(n, device=dev)
    W.fill_gradients(wl, 0, g)
    W.init_weights(wl, w)
    flags = B.MODE_EF
    if variant == "deferred":
        flags |= B.DEFERRED_RESIDUAL
    elif variant == "single_launch":
        flags |= B.FORCE_COOPERATIVE
    ctx = B.a2sgd_create(n, P, dev.index, flags)
    if variant == "dense_sync":
        call = lambda: B.a2sgd_dense_sync(ctx, w, g, wl.lr)
    elif variant == "bf16":
        g16 = torch.empty((P, g.stride(0)), dtype=torch.bfloat16, device=dev)[:, :n]
        g16.copy_(g)
        call = lambda: B.a2sgd_step_bf16(ctx, w, g16, e, wl.lr)
    elif variant == "momentum":
        mom = torch.zeros(n, device=dev)
        call = lambda: B.a2sgd_step_momentum(ctx, w, mom, g, e, wl.lr, 0.9, 1e-4)
    elif variant == "replicated":
        w_rep = B.padded_rows(P, n, dev)
        w_rep.copy_(w.expand(P, n))
        call = lambda: B.a2sgd_step(ctx, w_rep, g, e, wl.lr)
    elif variant == "segments":
        sizes = [sg.numel for sg in wl.segments]
        gs = [[t.clone() for t in torch.split(g[p], sizes)] for p in range(P)]
        es = [[t.clone() for t in torch.split(e[p], sizes)] for p in range(P)]
        ws = [t.clone() for t in torch.split(w, sizes)]
        plan = B.a2sgd_segments_create(ctx, gs, es, ws)
        call = lambda: B.a2sgd_step_segments(ctx, plan, wl.lr)
    else:  # deferred, single_launch, misaligned: the step entry point on that context / layout
        call = lambda: B.a2sgd_step(ctx, w, g, e, wl.lr)
    for _ in range(max(3, warmup)):
        call()
    torch.cuda.synchronize(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        call()
    ev1.record()
    torch.cuda.synchronize(dev)
    return ev0.elapsed_time(ev1) / steps


# ----------------------------------------------------------------------------- device arm
def max_over_ranks(ms: float, dist, device) -> float:
    """Every rank contributes its own device-timed milliseconds; all get the maximum."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(n_model: int, n_replicas: int, ms_per_step: float) -> float:
    """Model parameters per second summed over the independent replicas."""
    return n_replicas * n_model / (ms_per_step * 1e-3)


def spread(samples) -> dict:
    """median / min / max of a list of per-step (or per-launch) milliseconds."""
    xs = sorted(float(x) for x in samples)
    if not xs:
        return {"n": 0}
    mid = len(xs) // 2
    med = xs[mid] if len(xs) % 2 else 0.5 * (xs[mid - 1] + xs[mid])
    return {"median": med, "min": xs[0], "max": xs[-1], "n": len(xs)}


def host_description() -> dict:
    """Core count and CPU model of the box the oracle is timed on."""
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except AttributeError:
        usable = os.cpu_count()
    return {"nproc": os.cpu_count(), "usable_cores": usable, "cpu_model": model}


def time_workload(wl, steps, warmup, dev, *, with_roofline=True, with_next_rows=True, with_e2e=True, dist=None,
                  row_stride=None):
    """Runs the timed regions for one workload on this rank's GPU.  Returns a dict of results.
    ``row_stride`` overrides the 128-byte aligned row layout (e.g. n + 1: every row at a different
    4-byte phase, which takes the general-alignment kernels)."""
    import torch
    from paper_2006_07405_b200 import binding as B
    from paper_2006_07405_b200 import workloads as W

    n, P = wl.n, wl.P
    torch.cuda.set_device(dev)
    if row_stride is None:
        # rows start 128-byte aligned (row stride = n rounded up to 32 elements)
        g = B.padded_rows(P, n, dev)
        e = B.padded_rows(P, n, dev, fill=0.0)
    else:
        g = torch.empty((P, row_stride), device=dev)[:, :n]
        e = torch.zeros((P, row_stride), device=dev)[:, :n]
    w = torch.empty(n, device=dev)
    W.fill_gradients(wl, 0, g)
    W.init_weights(wl, w)
    ctx = B.a2sgd_create(n, P, dev.index, B.MODE_EF)
    info = B.a2sgd_launch_info(ctx, shared_w=True)
    launches_per_step = 1 if info["single_launch"] else 2

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(max(warmup, 3)):
        B.a2sgd_step(ctx, w, g, e, wl.lr)
    barrier()
    # A step of a few microseconds is bound by host launch overhead: replay it from a CUDA graph
    # (chunks of `chunk` steps, K = reps * chunk exactly).
    graph, chunk = None, 1
    if n * P < (1 << 23):
        chunk = max(d for d in range(1, 51) if steps % d == 0)
        try:
            side = torch.cuda.Stream(dev)
            side.wait_stream(torch.cuda.current_stream(dev))
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for _ in range(chunk):
                        B.a2sgd_step(ctx, w, g, e, wl.lr, stream=side)
            torch.cuda.current_stream(dev).wait_stream(side)
            graph.replay()
        except Exception as ex:  # capture refused: time eager launches instead
            graph, chunk = None, 1
            sys.stderr.write(f"CUDA graph capture failed ({ex}); timing eager launches\n")
        barrier()
    # One event before every step (or graph replay) and one after the last: the K steps are timed
    # as one region (first to last event); the events in between give the spread.
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps // chunk + 1)]
    wall0 = time.time()
    for i in range(steps // chunk):
        marks[i].record()
        if graph is not None:
            graph.replay()
        else:
            B.a2sgd_step(ctx, w, g, e, wl.lr)
    marks[-1].record()
    barrier()
    wall1 = time.time()
    ms = max_over_ranks(marks[0].elapsed_time(marks[-1]), dist, dev)
    per_step = [marks[i].elapsed_time(marks[i + 1]) / chunk for i in range(len(marks) - 1)]
    res = {"ms_total": ms, "ms_per_step": ms / steps, "launches": launches_per_step * steps,
           "step_ms_spread": spread(per_step),
           "launch_info": info, "wall": (wall0, wall1),
           "launch_mode": f"CUDA graph of {chunk} steps" if graph is not None else "eager"}
    del graph
    *_, status = B.a2sgd_read_stats(ctx)
    res["device_status"] = status

    if with_roofline:
        # the two kernels of a step each timed alone, in the launch configuration a2sgd_step uses
        lm = torch.zeros((P, 2), device=dev)
        gm = torch.zeros(2, device=dev)
        k_steps = max(5, min(steps, 200))
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(3 * k_steps)]
        for i in range(k_steps):
            evs[3 * i].record()
            B.a2sgd_encode(ctx, g, e, lm)
            B.a2sgd_global_average(ctx, lm, gm)
            evs[3 * i + 1].record()
            B.a2sgd_decode_update(ctx, w, g, e, lm, gm, wl.lr)
            evs[3 * i + 2].record()
        torch.cuda.synchronize(dev)
        enc = [evs[3 * i].elapsed_time(evs[3 * i + 1]) for i in range(k_steps)]
        dec = [evs[3 * i + 1].elapsed_time(evs[3 * i + 2]) for i in range(k_steps)]
        res["encode_ms"] = sum(enc) / k_steps
        res["decode_ms"] = sum(dec) / k_steps
        res["encode_ms_spread"] = spread(enc)
        res["decode_ms_spread"] = spread(dec)

    if with_next_rows:
        # rows beyond the core step: the dense synchronisation step (Algorithm 1 lines 9-10), the
        # deferred-residual and 16-bit-gradient forms, and the step over a segment list
        k_steps = max(5, min(steps, 50))
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(2)]

        def timed(call):
            for _ in range(3):
                call()
            evs[0].record()
            for _ in range(k_steps):
                call()
            evs[1].record()
            torch.cuda.synchronize(dev)
            return evs[0].elapsed_time(evs[1]) / k_steps

        res["dense_sync_ms"] = timed(lambda: B.a2sgd_dense_sync(ctx, w, g, wl.lr))
        if g.stride(0) % 8 == 0:
            dctx = B.a2sgd_create(n, P, dev.index, B.MODE_EF | B.DEFERRED_RESIDUAL)
            res["step_deferred_ms"] = timed(lambda: B.a2sgd_step(dctx, w, g, e, wl.lr))
            B.a2sgd_materialize_err(dctx, e)
            torch.cuda.synchronize(dev)
            dctx.destroy()
        actx = B.a2sgd_create(n, P, dev.index, B.MODE_ALG1)
        res["step_alg1_ms"] = timed(lambda: B.a2sgd_step(actx, w, g, None, wl.lr))
        actx.destroy()
        mom = torch.zeros(n, device=dev)
        res["step_momentum_ms"] = timed(lambda: B.a2sgd_step_momentum(ctx, w, mom, g, e, wl.lr, 0.9, 1e-4))
        del mom
        g16 = torch.empty((P, g.stride(0)), dtype=torch.bfloat16, device=dev)[:, :n]
        g16.copy_(g)
        res["step_bf16_ms"] = timed(lambda: B.a2sgd_step_bf16(ctx, w, g16, e, wl.lr))
        del g16
        torch.cuda.empty_cache()
        free_b, _ = torch.cuda.mem_get_info(dev)
        if hasattr(wl, "segments") and free_b > (2 * P + 1) * n * 4 * 1.1:
            sizes = [sg.numel for sg in wl.segments]
            gs = [[t.clone() for t in torch.split(g[p], sizes)] for p in range(P)]
            es = [[t.clone() for t in torch.split(e[p], sizes)] for p in range(P)]
            ws = [t.clone() for t in torch.split(w, sizes)]
            plan = B.a2sgd_segments_create(ctx, gs, es, ws)
            res["step_segments_ms"] = timed(lambda: B.a2sgd_step_segments(ctx, plan, wl.lr))
            res["step_segments_per_tensor_ms"] = timed(lambda: B.a2sgd_step_segments_per_tensor(ctx, plan, wl.lr))
            plan.destroy()
            del gs, es, ws, plan
            torch.cuda.empty_cache()

    if with_e2e:
        # every rank of the node holds its own host copy of the step's gradients: leave the leg out
        # (and say so) rather than exhaust host memory when N ranks x P*n*4 bytes do not fit
        try:
            import psutil
            host_free = psutil.virtual_memory().available
        except Exception:
            host_free = None
        ranks_here = int(os.environ.get("LOCAL_WORLD_SIZE", "1"))
        fits = not (host_free is not None and 1.25 * ranks_here * P * n * 4 > host_free)
        if dist is not None:   # one decision for all ranks: the leg contains collectives
            flag = torch.tensor([1.0 if fits else 0.0], device=dev, dtype=torch.float64)
            dist.all_reduce(flag, op=dist.ReduceOp.MIN)
            fits = bool(flag.item() > 0.5)
        if not fits:
            res["e2e_skipped"] = (f"{ranks_here} rank(s) x {P * n * 4 / 1e9:.1f} GB of host gradients do not fit in "
                                  f"{(host_free or 0) / 1e9:.0f} GB of free host memory")
            with_e2e = False
    if with_e2e:
        pinned = True
        try:
            g_host = torch.empty((P, n), pin_memory=True)
        except Exception as ex:
            sys.stderr.write(f"pinned allocation of {P * n * 4 / 1e9:.1f} GB failed ({ex}); pageable host memory\n")
            g_host, pinned = torch.empty((P, n)), False
        g_host.copy_(g)
        means = torch.zeros(2 * P + 2).pin_memory()
        e2e_steps = max(2, min(steps, 10 if n * P < (1 << 30) else 3))
        for _ in range(2):
            B.a2sgd_step_host(ctx, w, g_host, g, e, wl.lr, means)
        barrier()
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(e2e_steps + 1)]
        for i in range(e2e_steps):
            marks[i].record()
            B.a2sgd_step_host(ctx, w, g_host, g, e, wl.lr, means)
        marks[-1].record()
        barrier()
        ms2 = max_over_ranks(marks[0].elapsed_time(marks[-1]), dist, dev)
        res["e2e_ms_per_step"] = ms2 / e2e_steps
        res["e2e_ms_spread"] = spread([marks[i].elapsed_time(marks[i + 1]) for i in range(e2e_steps)])
        res["e2e_steps"] = e2e_steps
        res["e2e_pinned"] = pinned
        res["h2d_bytes"] = P * n * 4
        res["d2h_bytes"] = (2 * P + 2) * 4
        del g_host
    ctx.destroy()
    del g, e, w
    torch.cuda.empty_cache()
    return res


def load_loop_for_clocks(wl, dev, seconds):
    """Keeps the same kernels running so the clock sampler sees the GPU under this load."""
    import torch
    from paper_2006_07405_b200 import binding as B
    from paper_2006_07405_b200 import workloads as W
    n, P = wl.n, wl.P
    g = B.padded_rows(P, n, dev)
    e = B.padded_rows(P, n, dev, fill=0.0)
    w = torch.zeros(n, device=dev)
    W.fill_gradients(wl, 0, g)
    ctx = B.a2sgd_create(n, P, dev.index, B.MODE_EF)
    per_sync = 50 if n * P < (1 << 30) else 5
    t0 = time.time()
    while time.time() - t0 < seconds:
        for _ in range(per_sync):
            B.a2sgd_step(ctx, w, g, e, wl.lr)
        torch.cuda.synchronize(dev)
    ctx.destroy()


def kernel_rooflines(wl, res, peak_gbs) -> dict:
    """Per-kernel roofline records (K1 encode-reduce, K3 decode/update) from the per-launch event
    times of ``time_workload``: algorithmic bytes / launch duration against the measured peak."""
    b = algorithmic_bytes_per_model_element(wl.P)
    out = {}
    for key, name in (("encode", "encode-reduce (K1) + stand-alone global-average launch"),
                      ("decode", "decode/update (K3)")):
        ms = res[f"{key}_ms"]
        achieved = b[key] * wl.n / (ms * 1e-3) / 1e9
        out[key] = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                    "frac": achieved / peak_gbs, "frac_of_8TBps": achieved / NOMINAL_HBM_GBS,
                    "algorithmic_bytes": b[key] * wl.n, "launch_ms": ms, "launch_ms_spread": res[f"{key}_ms_spread"]}
    return out


def summarise(wl, res, n_gpus, peak_gbs):
    b = algorithmic_bytes_per_model_element(wl.P)
    t = res["ms_per_step"] * 1e-3
    out = {"n": wl.n, "P": wl.P, "ms_per_step": res["ms_per_step"], "step_ms_spread": res["step_ms_spread"],
           "launch_mode": res["launch_mode"],
           "single_launch": res["launch_info"]["single_launch"],
           "model_params_per_s": n_gpus * wl.n / t, "worker_params_per_s": n_gpus * wl.n * wl.P / t,
           "step_GBps": b["step"] * wl.n / t / 1e9,
           "step_frac_of_8TBps": b["step"] * wl.n / t / 1e9 / NOMINAL_HBM_GBS,
           "step_frac_of_measured_peak": b["step"] * wl.n / t / 1e9 / peak_gbs}
    if "decode_ms" in res:
        out["roofline"] = kernel_rooflines(wl, res, peak_gbs)
    rows = next_rows_of(wl, res, peak_gbs)
    if rows:
        out["next_rows"] = rows
    return out


def next_rows_of(wl, res, peak_gbs) -> dict:
    b = algorithmic_bytes_per_model_element(wl.P)
    rows = {}
    if "dense_sync_ms" in res:
        bts = (4 * wl.P + 8) * wl.n
        rows["dense_sync (Algorithm 1 lines 9-10)"] = {
            "ms": res["dense_sync_ms"], "GBps": bts / (res["dense_sync_ms"] * 1e-3) / 1e9,
            "frac_of_measured_peak": bts / (res["dense_sync_ms"] * 1e-3) / 1e9 / peak_gbs,
            "bytes_per_model_element": 4 * wl.P + 8}
    if "step_segments_ms" in res:
        bts = b["step"] * wl.n
        rows["step over a segment list (one tensor per segment)"] = {
            "ms": res["step_segments_ms"], "GBps": bts / (res["step_segments_ms"] * 1e-3) / 1e9,
            "frac_of_8TBps": bts / (res["step_segments_ms"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "segments": len(wl.segments)}
    if "step_segments_per_tensor_ms" in res:
        bts = b["step"] * wl.n
        rows["step over a segment list, every tensor compressed on its own (2S floats per worker)"] = {
            "ms": res["step_segments_per_tensor_ms"], "GBps": bts / (res["step_segments_per_tensor_ms"] * 1e-3) / 1e9,
            "frac_of_8TBps": bts / (res["step_segments_per_tensor_ms"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "segments": len(wl.segments)}
    if "step_deferred_ms" in res:
        bts = (12 * wl.P + 8 + wl.P / 4) * wl.n
        rows["step, deferred-residual representation (opt-in, bit-identical results)"] = {
            "ms": res["step_deferred_ms"], "GBps_actual_bytes": bts / (res["step_deferred_ms"] * 1e-3) / 1e9,
            "model_params_per_s": wl.n / (res["step_deferred_ms"] * 1e-3),
            "bytes_per_model_element": 12 * wl.P + 8 + wl.P / 4,
            "speedup_vs_canonical_step": res["ms_per_step"] / res["step_deferred_ms"]}
    if "step_alg1_ms" in res:
        bts = (8 * wl.P + 8) * wl.n
        rows["step in ALG1 mode (Algorithm 1 as printed: same-iteration add-back, eps not stored)"] = {
            "ms": res["step_alg1_ms"], "GBps": bts / (res["step_alg1_ms"] * 1e-3) / 1e9,
            "frac_of_8TBps": bts / (res["step_alg1_ms"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "model_params_per_s": wl.n / (res["step_alg1_ms"] * 1e-3), "bytes_per_model_element": 8 * wl.P + 8}
    if "step_momentum_ms" in res:
        bts = (20 * wl.P + 16) * wl.n
        rows["step with momentum and weight decay (a2sgd_step_momentum)"] = {
            "ms": res["step_momentum_ms"], "GBps": bts / (res["step_momentum_ms"] * 1e-3) / 1e9,
            "frac_of_8TBps": bts / (res["step_momentum_ms"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "model_params_per_s": wl.n / (res["step_momentum_ms"] * 1e-3), "bytes_per_model_element": 20 * wl.P + 16}
    if "step_bf16_ms" in res:
        bts = (16 * wl.P + 8) * wl.n
        rows["step with bfloat16 gradients"] = {
            "ms": res["step_bf16_ms"], "GBps": bts / (res["step_bf16_ms"] * 1e-3) / 1e9,
            "frac_of_8TBps": bts / (res["step_bf16_ms"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "model_params_per_s": wl.n / (res["step_bf16_ms"] * 1e-3), "bytes_per_model_element": 16 * wl.P + 8}
    return rows


class DeviceTimer:
    """CUDA-event stopwatch on the current stream of ``dev``."""

    def __init__(self, dev):
        import torch
        self.torch, self.dev = torch, dev

    def mark(self):
        ev = self.torch.cuda.Event(enable_timing=True)
        ev.record()
        return ev

    def sync(self):
        self.torch.cuda.synchronize(self.dev)

    def ms(self, a, b):
        return a.elapsed_time(b)


class HostTimer:
    """Wall-clock stand-in with the same interface (CPU tests of the multi-rank protocol)."""

    def __init__(self, dev=None):
        self.dev = dev

    def mark(self):
        return time.perf_counter()

    def sync(self):
        pass

    def ms(self, a, b):
        return (b - a) * 1e3


def exchange_leg(sizes, make_case, dist, dev, steps, warmup, timer):
    """One worker per rank, as Algorithm 1 prints it: for every n in ``sizes`` and both exchanges
    of the two local means (all-gather + local fixed-order average; all-reduce + division), times
    the whole step (encode, exchange, decode/update) and the exchange alone, K calls each,
    bracketed by barriers, max over ranks.  ``make_case(n, exchange)`` returns (worker, step_call)
    where ``worker.exchange_means()`` is the exchange alone and ``step_call()`` one whole step."""
    def barrier():
        timer.sync()
        dist.barrier()
        timer.sync()

    out = {"workers": dist.get_world_size(), "payload_bytes_per_worker": 8, "sizes": {}}
    for n in sizes:
        row = {}
        for exchange in ("allgather", "allreduce"):
            worker, step_call = make_case(n, exchange)
            for _ in range(max(3, warmup)):
                step_call()
            barrier()
            t0 = timer.mark()
            for _ in range(steps):
                step_call()
            t1 = timer.mark()
            barrier()
            step_ms = max_over_ranks(timer.ms(t0, t1), dist, dev) / steps
            for _ in range(max(3, warmup)):
                worker.exchange_means()
            barrier()
            reps = max(steps, 50)
            t0 = timer.mark()
            for _ in range(reps):
                worker.exchange_means()
            t1 = timer.mark()
            barrier()
            ex_us = max_over_ranks(timer.ms(t0, t1), dist, dev) / reps * 1e3
            row[exchange] = {"ms_per_step": step_ms, "us_per_exchange": ex_us,
                             "worker_params_per_s": dist.get_world_size() * n / (step_ms * 1e-3)}
            worker.destroy()
        out["sizes"][str(n)] = row
    return out


def device_exchange_case(dev, lr):
    """make_case for exchange_leg on GPUs: DistributedA2SGD with seeded per-rank gradients."""
    import torch
    from paper_2006_07405_b200 import binding as B
    from paper_2006_07405_b200 import distributed as D

    def make(n, exchange):
        import torch.distributed as dist_mod
        gen = torch.Generator(device=dev).manual_seed(20060740 + dist_mod.get_rank())
        g = B.padded_rows(1, n, dev).normal_(0.0, 1e-3, generator=gen)
        e = B.padded_rows(1, n, dev, fill=0.0)
        w = torch.zeros(n, device=dev)
        worker = D.DistributedA2SGD(n, dev.index, B.MODE_EF, exchange=exchange)
        return worker, (lambda: worker.step(w, g, e, lr))
    return make


def pick_workload(name, scale_div, dev):
    """The requested workload, or the fallback when the device cannot hold its resident set."""
    import torch
    from paper_2006_07405_b200 import workloads as W
    wl = W.get_workload(name)
    if scale_div > 1:
        wl = W.scaled(wl, scale_div)
    note = None
    free_b, _ = torch.cuda.mem_get_info(dev)
    need = (2 * wl.P + 1) * wl.n * 4 * 1.05
    if need > free_b and name == DEFAULT_WORKLOAD and scale_div == 1:
        note = (f"{name} needs {need / 1e9:.0f} GB of device memory, {free_b / 1e9:.0f} GB free: "
                f"fell back to {FALLBACK_WORKLOAD}")
        wl = W.get_workload(FALLBACK_WORKLOAD)
    return wl, note


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations at N=1")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--exchange-leg", action="store_true",
                    help="under torchrun: run the one-worker-per-GPU exchange leg even with a single rank")
    ap.add_argument("--scale-div", type=int, default=1,
                    help="divide every tensor length of the workload (small cases for profiler captures)")
    ap.add_argument("--variant", default="step",
                    choices=["step", "dense_sync", "deferred", "bf16", "segments", "single_launch", "momentum",
                             "replicated", "misaligned"],
                    help="with --minimal: which entry point the bare loop calls")
    ap.add_argument("--minimal", action="store_true",
                    help="timed step loop only (for profiler captures): no e2e, no per-kernel loop, "
                         "no extra workloads, no clock load loop, no CPU baseline")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2006_07405_b200 import binding as B
    from paper_2006_07405_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the A2SGD path has no CPU fallback")
    from paper_2006_07405_b200 import build as cuda_build
    cuda_build.build()   # compiles only when the library is missing or older than its sources (atomic replace)
    B.lib()  # fails loudly if the CUDA library is still missing: there is no other path

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:   # launched by torchrun: same protocol at any N
        import torch.distributed as dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod
    n_gpus = world
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    wl, fallback_note = pick_workload(args.workload, args.scale_div, dev)
    peak_gbs, peak_src = measured_peak_gbs()
    steps, warmup = max(1, args.steps), max(3, args.warmup)

    if args.minimal and args.variant != "step":
        ms = run_variant(wl, args.variant, steps, warmup, dev)
        print(json.dumps({"variant": args.variant, "ms_per_call": ms, "steps": steps, "config": W.describe(wl),
                          "note": "minimal run for profiler captures"}), flush=True)
        return
    if args.minimal:
        res = time_workload(wl, steps, warmup, dev, with_roofline=False, with_next_rows=False, with_e2e=False,
                            dist=dist)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": n_gpus * wl.n / (res["ms_per_step"] * 1e-3), "unit": UNIT,
                              "ms_per_step": res["ms_per_step"], "steps": steps, "warmup": warmup,
                              "config": W.describe(wl), "note": "minimal run for profiler captures"}), flush=True)
        if dist is not None:
            dist.destroy_process_group()
        return
    sampler = ClockSampler(local_rank) if rank == 0 else None
    res = time_workload(wl, steps, warmup, dev, dist=dist)
    if rank == 0 and res["ms_total"] < 1500.0:
        load_loop_for_clocks(wl, dev, 1.5)
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["sampled_over"] = "timed region" if res["ms_total"] >= 1500.0 else \
            "timed region plus 1.5 s of the same step loop (timed region shorter than the sampling period allows)"

    extra = {}
    if rank == 0 and world == 1 and not args.no_extra and args.scale_div == 1:
        for name in ("c1_flat_1m", "c2_lstm_ptb", "c3_resnet50", "c4_vgg16", "c5_gpt2_xl"):
            if name == wl.name:
                continue
            w2 = W.get_workload(name)
            free_b, _ = torch.cuda.mem_get_info(dev)
            if (2 * w2.P + 1) * w2.n * 4 * 1.05 > free_b:
                extra[name] = {"skipped": "not enough free device memory"}
                continue
            k = 20 if w2.n > 10 ** 9 else (100 if w2.n > 10 ** 7 else 1000)
            r2 = time_workload(w2, k, 3, dev, with_e2e=False)
            extra[name] = summarise(w2, r2, 1, peak_gbs)
        # rows that are only 4-byte aligned, each at a different phase: the general-alignment kernels
        w2 = W.get_workload(FALLBACK_WORKLOAD)
        r2 = time_workload(w2, 100, 3, dev, with_e2e=False, with_next_rows=False, row_stride=w2.n + 1)
        extra[f"{w2.name}, rows misaligned (row stride n + 1, 32-bit coalesced accesses)"] = summarise(w2, r2, 1, peak_gbs)

    exchange = None
    if dist is not None and ((world > 1 and not args.no_extra) or args.exchange_leg):
        # the O(1) exchange between real GPUs (Algorithm 1 line 5), all-gather against all-reduce
        sizes = sorted({1 << 20, W.get_workload("c2_lstm_ptb").n, wl.n})
        exchange = exchange_leg(sizes, device_exchange_case(dev, wl.lr), dist, dev, steps, warmup, DeviceTimer(dev))
    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    b = algorithmic_bytes_per_model_element(wl.P)
    t = res["ms_per_step"] * 1e-3
    value = whole_job_value(wl.n, n_gpus, res["ms_per_step"])
    roofs = kernel_rooflines(wl, res, peak_gbs)
    traffic_per_el = NCU_DECODE_TRAFFIC_PER_ELEMENT.get(wl.P)
    config = dict(W.describe(wl), mode="EF", w_layout="one shared w", resident_GB=(2 * wl.P + 1) * wl.n * 4 / 1e9,
                  l2="inputs larger than L2: every step streams the whole resident set",
                  parallelism=f"{n_gpus} independent replica(s), no collective",
                  worker_params_per_s=n_gpus * wl.n * wl.P / t,
                  step_GBps=b["step"] * wl.n / t / 1e9,
                  step_frac_of_8TBps=b["step"] * wl.n / t / 1e9 / NOMINAL_HBM_GBS,
                  step_frac_of_measured_peak=b["step"] * wl.n / t / 1e9 / peak_gbs,
                  step_ms_spread=res["step_ms_spread"],
                  bytes_per_model_element=b, launch=res["launch_info"], launch_mode=res["launch_mode"],
                  row_stride="n rounded up to 32 elements (rows start 128-byte aligned)",
                  encode_ms=res["encode_ms"], decode_ms=res["decode_ms"],
                  device_status=res["device_status"])
    if fallback_note:
        config["fallback"] = fallback_note
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": n_gpus, "steps": steps, "warmup": warmup,
        "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": config,
        "gpu_launches": res["launches"],
        "clocks": clocks,
        "e2e": ({"value": n_gpus * wl.n / (res["e2e_ms_per_step"] * 1e-3), "unit": UNIT,
                 "h2d_bytes_per_step": res["h2d_bytes"], "d2h_bytes_per_step": res["d2h_bytes"],
                 "ms_per_step": res["e2e_ms_per_step"], "ms_spread": res["e2e_ms_spread"], "steps": res["e2e_steps"],
                 "host_memory": "pinned" if res["e2e_pinned"] else "pageable (pinned allocation failed)",
                 "api": "a2sgd_step_host (pinned host gradients in, 2P+2 means out)"}
                if "e2e_ms_per_step" in res else
                {"value": None, "unit": UNIT, "h2d_bytes_per_step": wl.P * wl.n * 4, "d2h_bytes_per_step": (2 * wl.P + 2) * 4,
                 "skipped": res.get("e2e_skipped", "not run")}),
        "roofline": dict(roofs["decode"], peak_source=peak_src,
                         traffic=traffic_per_el * wl.n if traffic_per_el else None,
                         traffic_source="ncu dram__bytes read+write per model element of a smaller capture of the "
                                        "same kernel (profiles/), scaled by n" if traffic_per_el else None,
                         encode_kernel=roofs["encode"]),
    }
    rows = next_rows_of(wl, res, peak_gbs)
    if rows:
        line["next_rows"] = rows
    if extra:
        line["other_workloads"] = extra
    if exchange:
        line["exchange_between_gpus"] = exchange
    if not args.no_cpu_baseline and world == 1:
        cb = oracle_sample_rate(wl, 10.0, all_cores=True)
        line["cpu_baseline"] = dict({k: v for k, v in cb.items() if not k.startswith("_")}, host=host_description())
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
