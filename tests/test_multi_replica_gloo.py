"""Host-side logic of the multi-GPU benchmark mode, on CPU with gloo (world size 2).

The measured path has no exchange between GPUs, so N GPUs run N independent replicas; what
the ranks share is only the timing protocol: barrier, max over ranks of the device time, and
rank 0 reporting the whole-job value."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import torch
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
    rank = dist.get_rank()
    dist.barrier()
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
    assert ms == 15.0, ms
    value = bench.whole_job_value(1000, dist.get_world_size(), ms)
    assert abs(value - 2 * 1000 / 15e-3) < 1e-6
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


def test_max_over_ranks_and_whole_job_value_world_size_2(tmp_path):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {r} ok" in out


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.algorithmic_bytes_per_model_element(4) == {"encode": 32, "decode": 56, "step": 88}
    assert bench.algorithmic_bytes_per_model_element(8)["step"] == 168
    assert bench.algorithmic_bytes_per_model_element(1)["step"] == 28


def test_reference_arm_json_line_has_the_contract_keys():
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "c1_flat_1m", "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["value"] > 0 and line["config"]["workload"] == "c1_flat_1m"


EXCHANGE_WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import torch
    import torch.distributed as dist
    import bench
    from paper_2006_07405_b200 import distributed as D
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
    rank = dist.get_rank()

    class FakeWorker:
        # the exchange itself is real (gloo); the kernels around it are not needed for the protocol
        def __init__(self, exchange):
            self.exchange, self.calls, self.destroyed = exchange, 0, False
            self.local_means = torch.tensor([[1.0 + rank, 2.0 + rank]])
        def exchange_means(self):
            self.calls += 1
            if self.exchange == "allgather":
                got = D.exchange_local_means(self.local_means)
                assert got.tolist() == [[1.0, 2.0], [2.0, 3.0]]
            else:
                assert D.sum_local_means(self.local_means).tolist() == [3.0, 5.0]
        def destroy(self):
            self.destroyed = True

    made = []
    def make_case(n, exchange):
        w = FakeWorker(exchange)
        made.append(w)
        return w, w.exchange_means
    out = bench.exchange_leg([1000, 2000], make_case, dist, torch.device("cpu"), steps=4, warmup=1,
                             timer=bench.HostTimer())
    assert out["workers"] == 2 and out["payload_bytes_per_worker"] == 8
    assert sorted(out["sizes"]) == ["1000", "2000"]
    for n, row in out["sizes"].items():
        for ex in ("allgather", "allreduce"):
            r = row[ex]
            assert r["ms_per_step"] > 0 and r["us_per_exchange"] > 0
            assert abs(r["worker_params_per_s"] - 2 * int(n) / (r["ms_per_step"] * 1e-3)) < 1e-3 * r["worker_params_per_s"]
    assert len(made) == 4 and all(w.destroyed for w in made)
    # warm-up 3 + 4 timed steps, then warm-up 3 + 50 timed exchanges
    assert all(w.calls == 3 + 4 + 3 + 50 for w in made), [w.calls for w in made]
    # both ranks hold the same (max over ranks) figures
    flat = torch.tensor([out["sizes"][n][ex][k] for n in sorted(out["sizes"]) for ex in ("allgather", "allreduce")
                         for k in ("ms_per_step", "us_per_exchange")], dtype=torch.float64)
    other = [torch.zeros_like(flat) for _ in range(2)]
    dist.all_gather(other, flat)
    assert torch.equal(other[0], other[1])
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


def test_exchange_leg_protocol_world_size_2(tmp_path):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(EXCHANGE_WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {r} ok" in out


def test_bench_line_helpers():
    """The pure helpers behind the JSON line: spread of per-step times, per-kernel roofline records
    (algorithmic bytes / launch time against the peak) and the rows beyond the plain step."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2006_07405_b200 import workloads as W
    s = bench.spread([3.0, 1.0, 2.0, 10.0])
    assert s == {"median": 2.5, "min": 1.0, "max": 10.0, "n": 4}
    assert bench.spread([]) == {"n": 0}
    wl = W.get_workload("c4_vgg16")
    res = {"encode_ms": 0.6, "decode_ms": 1.1, "encode_ms_spread": s, "decode_ms_spread": s}
    roofs = bench.kernel_rooflines(wl, res, 6529.7)
    dec = roofs["decode"]
    assert dec["bound"] == "hbm" and dec["unit"] == "GB/s" and dec["peak"] == 6529.7
    assert dec["algorithmic_bytes"] == (12 * wl.P + 8) * wl.n
    assert abs(dec["achieved"] - dec["algorithmic_bytes"] / 1.1e-3 / 1e9) < 1e-6
    assert abs(dec["frac"] - dec["achieved"] / 6529.7) < 1e-12
    assert roofs["encode"]["algorithmic_bytes"] == 8 * wl.P * wl.n
    rows = bench.next_rows_of(wl, {"ms_per_step": 1.7, "dense_sync_ms": 0.46, "step_momentum_ms": 1.9,
                                   "step_alg1_ms": 0.8, "step_bf16_ms": 1.45}, 6529.7)
    assert len(rows) == 4
    mom = rows["step with momentum and weight decay (a2sgd_step_momentum)"]
    assert mom["bytes_per_model_element"] == 20 * wl.P + 16
    assert set(bench.host_description()) == {"nproc", "usable_cores", "cpu_model"}
    assert bench.NCU_DECODE_TRAFFIC_PER_ELEMENT[4] < 12 * 4 + 8 < bench.NCU_DECODE_TRAFFIC_PER_ELEMENT[8]
