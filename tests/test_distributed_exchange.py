"""One worker per process: the exchange of the two local means between ranks.

The CPU test covers the exchange helpers alone (gloo, world size 2).  The GPU test runs two
worker processes that share cuda:0 (their kernels never wait on one another: the exchange is a
host-side collective between launches) through three compressed iterations and the dense
synchronisation step, and compares each worker's replica with the oracle's P = 2 result."""
import os
import socket
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_ranks(script_text, tmp_path, world=2, timeout=300):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(script_text.format(root=ROOT, port=port, world=world))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(world)]
    outs = [p.communicate(timeout=timeout)[0] for p in procs]
    for r, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, f"rank {r}:\n{out}"
        assert f"rank {r} ok" in out, out


CPU_WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, {root!r})
    import torch
    import torch.distributed as dist
    from paper_2006_07405_b200 import distributed as D
    rank = int(sys.argv[1])
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size={world})
    lm = torch.tensor([[1.0 + rank, 10.0 * (rank + 1)]])
    gathered = D.exchange_local_means(lm)
    assert gathered.tolist() == [[1.0, 10.0], [2.0, 20.0]], gathered
    sums = D.sum_local_means(lm)
    assert sums.dtype == torch.float64 and sums.tolist() == [3.0, 30.0], sums
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


def test_exchange_helpers_world_size_2_gloo(tmp_path):
    _run_ranks(CPU_WORKER, tmp_path)


GPU_WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, {root!r})
    sys.path.insert(0, {root!r} + "/tests")
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2006_07405_b200 import binding as B, distributed as D, workloads as W
    from parity_util import assert_means, assert_state, count_outliers, tau_w
    rank = int(sys.argv[1])
    world = {world}
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    wl = W.scaled(W.get_workload("c2_lstm_ptb"), 64)
    n = wl.n
    for exchange, mode in (("allgather", B.MODE_EF), ("allreduce", B.MODE_EF), ("allgather", B.MODE_ALG1)):
        all_g = torch.empty((4, n), device="cuda")           # every rank generates the same 4 rows, uses its own
        w = torch.empty(n, device="cuda")
        W.init_weights(wl, w)
        e = torch.zeros((1, n), device="cuda")
        w_ref = np.tile(w.cpu().numpy(), (world, 1))
        e_ref = np.zeros((world, n), np.float32)
        worker = D.DistributedA2SGD(n, 0, mode, exchange=exchange)
        for step in range(3):
            W.fill_gradients(wl, step, all_g)
            g = all_g[rank:rank + 1]
            worker.step(w, g, e, wl.lr)
            lm_ref, gm_ref, _ = oracle.step(w_ref, all_g[:world].cpu().numpy(), e_ref, wl.lr, mode=mode)
            assert_means(worker.local_means.cpu().numpy()[0], lm_ref[rank])
            assert_means(worker.global_means.cpu().numpy(), gm_ref)
            assert_state(w.cpu().numpy(), w_ref[rank], e.cpu().numpy()[0], e_ref[rank], gm_ref,
                         f"{{exchange}} mode {{mode}} step {{step}}", max_outliers=0 if step == 0 else 2)
        W.fill_gradients(wl, 3, all_g)
        worker.dense_sync(w, all_g[rank:rank + 1], wl.lr)
        oracle.dense_sync(w_ref, all_g[:world].cpu().numpy(), wl.lr)
        assert count_outliers(w.cpu().numpy(), w_ref[rank], tau_w(w_ref[rank])) <= 2
        worker.destroy()
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""")


@pytest.mark.gpu
def test_two_worker_processes_match_oracle(tmp_path):
    _run_ranks(GPU_WORKER, tmp_path, timeout=600)
