"""Rank bookkeeping of the benchmark on CPU: gloo, world size 2, rendezvous on 127.0.0.1."""

import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # rank r measured (10 + 5r) ms in total and (4 + r) ms in saves
    got = bench.max_over_ranks([10.0 + 5 * rank, 4.0 + rank], torch.device("cpu"), world)
    q.put((rank, got))
    dist.barrier()
    dist.destroy_process_group()


def test_times_are_the_maximum_over_ranks_and_throughput_sums():
    import torch.multiprocessing as mp

    sys.path.insert(0, ROOT)
    import bench

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert out[0] == out[1] == [15.0, 5.0]
    # two replicas that each scanned 8 GB in at most 5 ms: 3.2 TB/s for the job
    assert bench.job_throughput_gbs(2, 8e9, 5.0) == pytest.approx(3200.0)
    assert bench.max_over_ranks([1.5, 2.5], None, 1) == [1.5, 2.5]


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--n-elems", str(1 << 20)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["gpu_launches"] == 0
    assert rec["metric"] == bench_metric() and rec["unit"] == "GB/s" and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] == 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["config"]["n_elems"] == 1 << 20


def bench_metric():
    sys.path.insert(0, ROOT)
    import bench

    return bench.METRIC


def test_save_byte_model():
    sys.path.insert(0, ROOT)
    import bench

    n = 1 << 30
    assert bench.save_bytes(n, 0) == 2 * n * 4
    assert bench.save_bytes(n, n // 2) == (2 * n + 3 * (n // 2)) * 4  # (2 + 3r) N s
    assert bench.save_bytes(n, n) == 4 * n * 4  # a full checkpoint is one fused pass: no second read
