#!/usr/bin/env python
"""Benchmark of the SCAR checkpoint-and-recover pass on the CNN-scale parameter set.

One step = the whole hot path over one synthetic parameter set of 2**30 float32 elements in
4096-element blocks: a prioritized save at every r of the sweep (0.01, 0.1, 0.5, 1.0; the running
checkpoint is put back to its pristine state before each, outside the timed region), the read-only
full-recovery perturbation norm, and a partial recovery of one of eight shards.  Every timed call is
bracketed by CUDA events on the stream the library launches on; a step's time is the sum of its
timed calls.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its own
GPU: the method's pass over one device's parameters needs no exchange, so there is no collective on
the data path; the reported value is the sum over ranks divided by the slowest rank's time.

``--impl reference`` times the plain CPU oracle (``oracle/``) on the host cores over a bounded
sample of the same parameter set, with the same metric.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

R_SWEEP = (0.01, 0.1, 0.5, 1.0)
N_ELEMS = 1 << 30
BLOCK = 4096
ELEM = 4
METRIC = "prioritized-checkpoint GB/s scanned"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def recorded_traffic(n_elems: int):
    """DRAM bytes per k_block_scores launch from the last ncu capture, scaled to n_elems; None when there
    is no capture or the kernel sources changed after it was taken."""
    import hashlib

    pkg = os.path.join(ROOT, "paper_1810_07354_b200")
    try:
        with open(os.path.join(pkg, "ncu_traffic.json")) as f:
            rec = json.load(f)["k_block_scores"]
        h = hashlib.sha256()
        for name in ("geom.cuh", "block_pass.cuh"):
            with open(os.path.join(pkg, "csrc", name), "rb") as f:
                h.update(f.read())
        if h.hexdigest() != rec["src_sha256"]:
            return None
        return rec["dram_bytes_per_launch"] * (n_elems / rec["n_elems"])
    except Exception:
        return None


def save_bytes(n_elems: int, payload_elems: int) -> int:
    """Algorithmic bytes of one save: both streams read once, the selected blocks read again and written twice."""
    return 2 * n_elems * ELEM + 3 * payload_elems * ELEM


# ----------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background."""

    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str, period_ms: int = 50):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False).name
        self.f = open(self.path, "w")
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", gpu_uuid, f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", str(period_ms)],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self, t0: float, t1: float) -> dict:
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.p.kill()
        self.f.close()
        rows = []
        from datetime import datetime

        with open(self.path) as f:
            for line in f:
                c = [s.strip() for s in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    ts = datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(c[1]), float(c[2]), float(c[3]), c[4:9]))
                except ValueError:
                    continue
        os.unlink(self.path)
        inside = [r for r in rows if t0 - 0.05 <= r[0] <= t1 + 0.05] or rows
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            for name, val in zip(names, r[4][1:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median([r[1] for r in inside])), "sm_max_mhz": inside[0][2],
                "power_w_max": max(r[3] for r in inside), "samples": len(inside), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- CPU oracle legs


def oracle_step(x, z, boff, lost_blocks, timers):
    """One step of the hot path on the oracle; returns seconds spent in saves and in total."""
    import oracle

    t_save = 0.0
    t0 = time.perf_counter()
    for r in R_SWEEP:
        t = time.perf_counter()
        oracle.priority_save(x, z, boff, r=r)
        t_save += time.perf_counter() - t
    t = time.perf_counter()
    oracle.perturbation_norm(x, z, boff, None)
    oracle.recover_partial(x, z, boff, lost_blocks)
    timers["recover_s"] = timers.get("recover_s", 0.0) + time.perf_counter() - t
    return t_save, time.perf_counter() - t0


def run_reference(args):
    """The oracle as it stands, single-threaded, on a bounded sample of the CNN-scale set."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from workloads import block_offsets, make_workload

    # One oracle step over 2**26 elements takes about 5 s; shrink the sample so that warm-up plus
    # timed steps stay within a couple of minutes.
    n = 1 << 26
    while n > (1 << 22) and 5.0 * (n / (1 << 26)) * (args.steps + args.warmup) > 120.0:
        n >>= 1
    n = max(BLOCK, min(n, args.n_elems))
    w = make_workload("cnn", n_elems=n, block_elems=BLOCK)
    boff = block_offsets(w.geom)
    lost = oracle.expand_shards(w.n_blocks, w.lost_shards)
    timers = {}
    for _ in range(args.warmup):
        oracle_step(w.x, w.z, boff, lost, timers)
    t_save = t_all = 0.0
    for _ in range(args.steps):
        a, b = oracle_step(w.x, w.z, boff, lost, timers)
        t_save += a
        t_all += b
    value = len(R_SWEEP) * 2 * n * ELEM * args.steps / t_save / 1e9
    sample = f"first {n} of {N_ELEMS} elements ({w.n_blocks} blocks), numpy-generated with the same recipe"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cnn-scale fp32 vector, block 4096, r sweep 0.01/0.1/0.5/1.0 + full norm + "
                               "recovery of 1 of 8 shards", "n_elems": n, "sample_of": N_ELEMS},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(x_dev, z_dev, lost_shards):
    """Times the oracle on a prefix of the device-resident workload (copied to the host)."""
    import oracle

    n = min(x_dev.numel(), 1 << 30)
    nb = n // BLOCK
    x = x_dev[:n].cpu().numpy()
    z = z_dev[:n].cpu().numpy()
    boff = oracle.layout_offsets(n, 0, BLOCK)
    lost = oracle.expand_shards(nb, lost_shards)
    t_save, _ = oracle_step(x, z, boff, lost, {})
    return {"value": len(R_SWEEP) * 2 * n * ELEM / t_save / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"one step on {n} of {N_ELEMS} elements ({nb} blocks) of the same buffers, "
                      f"single thread, {t_save:.1f} s in saves"}


# ----------------------------------------------------------------------------- GPU arm


def max_over_ranks(values, device, world):
    """Element-wise maximum of per-rank device times: the job is as slow as its slowest replica."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist

    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput_gbs(world, bytes_per_rank, max_ms):
    """Whole-job GB/s: every rank moved bytes_per_rank in at most max_ms."""
    return world * bytes_per_rank / (max_ms * 1e-3) / 1e9


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_1810_07354_b200 import api
    from workloads.configs import make_cnn_device

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the library")
    api.load_library()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    n = args.n_elems
    geom, z0, x0, lost_shards = make_cnn_device(n, BLOCK, seed=4 + rank, device=dev)
    x = x0.clone()
    ck = api.ScarCheckpoint(x, n_shards=8, block_elems=BLOCK)
    ctx = ck.ctx
    nb = ck.n_blocks
    shard_lo = int(np.flatnonzero(lost_shards)[0]) * (nb // 8) * BLOCK
    shard_hi = shard_lo + (nb // 8) * BLOCK
    lost_elems = shard_hi - shard_lo

    z_lib = ck.views()["z"]  # the library's running checkpoint, aliased (no copy)
    flush = torch.empty(64 << 20, dtype=torch.float32, device=dev)  # 256 MiB, larger than the 126 MB L2

    def reset_checkpoint():
        """Pristine running checkpoint, then an L2 flush; plain torch copies, outside every timed interval."""
        z_lib.copy_(z0)
        flush.zero_()

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def one_step(rec):
        """Runs one step; appends (kind, start_event, end_event) triples to rec."""
        for r in R_SWEEP:
            reset_checkpoint()
            a, b = ev(), ev()
            a.record()
            ck.priority_save(r, sync=False)
            b.record()
            rec.append((("save", r), a, b))
        a, b = ev(), ev()
        a.record()
        ck.perturbation_norm(None, sync=False)
        b.record()
        rec.append((("norm", None), a, b))
        a, b = ev(), ev()
        a.record()
        ck.recover_partial(lost_shards, sync=False)
        b.record()
        rec.append((("recover", None), a, b))
        x[shard_lo:shard_hi].copy_(x0[shard_lo:shard_hi])  # put the live parameters back (not timed)
        flush.zero_()

    for _ in range(args.warmup):
        one_step([])
    barrier()

    # payload sizes per r (data dependent but fixed for this workload)
    payload_elems = {}
    for r in R_SWEEP:
        reset_checkpoint()
        payload_elems[r] = int(ck.priority_save(r).payload_elems)
    barrier()

    # ---- timed region: K steps, device-timed
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid)) if rank == 0 else None
    launches0 = api.scar_ckpt_launch_count(ctx)
    rec = []
    barrier()
    w0 = time.time()
    for _ in range(args.steps):
        one_step(rec)
    barrier()
    w1 = time.time()
    launches = api.scar_ckpt_launch_count(ctx) - launches0
    clocks = sampler.stop(w0, w1) if sampler else None

    t = {}
    for (kind, r), a, b in rec:
        t.setdefault((kind, r), []).append(a.elapsed_time(b))
    tot_ms = sum(sum(v) for v in t.values())
    save_ms = sum(sum(v) for (kind, _), v in t.items() if kind == "save")
    tot_ms, save_ms = max_over_ranks([tot_ms, save_ms], dev, world)

    # ---- dominant kernel (block scores) timed live through the library's own stream events
    api.scar_ckpt_profile(ctx, True)
    phase = {r: [] for r in R_SWEEP}
    rec_phase = []
    for _ in range(min(args.steps, 10)):
        for r in R_SWEEP:
            reset_checkpoint()
            ck.priority_save(r, sync=False)
            phase[r].append(api.scar_ckpt_profile_read(ctx))
        ck.recover_partial(lost_shards, sync=False)
        rec_phase.append(api.scar_ckpt_profile_read(ctx))
        x[shard_lo:shard_hi].copy_(x0[shard_lo:shard_hi])
    api.scar_ckpt_profile(ctx, False)
    score_ms = float(np.mean([p[0] for r in R_SWEEP for p in phase[r]]))

    if rank != 0:
        barrier()
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = hbm_peak()
    scanned = 2 * n * ELEM
    value = job_throughput_gbs(world, len(R_SWEEP) * scanned * args.steps, save_ms)
    per_r = {}
    for r in R_SWEEP:
        ms = float(np.median(t[("save", r)]))
        by = save_bytes(n, payload_elems[r])
        ph = np.median(np.array(phase[r]), axis=0)
        per_r[str(r)] = {"save_ms": ms, "scanned_gbs": scanned / ms / 1e6, "algorithmic_gbs": by / ms / 1e6,
                         "frac_of_measured_peak": by / ms / 1e6 / peak, "frac_of_8tbs": by / ms / 1e6 / 8000.0,
                         "blocks_per_s": nb / (ms * 1e-3), "payload_elems": payload_elems[r],
                         "phase_ms": {"scores": float(ph[0]), "select": float(ph[1]), "pack": float(ph[2])}}
    norm_ms = float(np.median(t[("norm", None)]))
    rec_ms = float(np.median(t[("recover", None)]))
    rph = np.median(np.array(rec_phase), axis=0)
    achieved = scanned / (score_ms * 1e-3) / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": tot_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "cnn-scale fp32 vector, block 4096, r sweep 0.01/0.1/0.5/1.0 + full norm + "
                               "recovery of 1 of 8 shards", "n_elems": n, "n_blocks": nb, "r_sweep": list(R_SWEEP),
                   "l2": "inputs larger than L2 (8 GiB scanned per save); L2 also flushed by a 256 MiB write "
                         "after every untimed state reset",
                   "value_is": "sum over the r sweep of 2*N*4 bytes / sum of save times",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "save_ms_per_step": save_ms / args.steps,
        "per_r": per_r,
        "perturbation_norm": {"ms": norm_ms, "gbs": scanned / norm_ms / 1e6},
        "partial_recovery": {"ms": rec_ms, "gbs": 3 * lost_elems * ELEM / rec_ms / 1e6, "lost_elems": lost_elems,
                             "phase_ms": {"restore": float(rph[3]), "reduce": float(rph[4])}},
        "roofline": {"bound": "hbm", "kernel": "k_block_scores", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"of {peak_kind}", "traffic": recorded_traffic(n),
                     "bytes_per_launch": scanned, "ms_per_launch": score_ms},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "wall_s_timed_region": w1 - w0,
    }

    if not args.no_e2e:
        line["e2e"] = run_e2e(api, ck, x, x0, z0, lost_shards, shard_lo, shard_hi, n, nb, world)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(x0, z0, lost_shards)
    print(json.dumps(line))
    barrier()
    if world > 1:
        dist.destroy_process_group()


def run_e2e(api, ck, x, x0, z0, lost_shards, shard_lo, shard_hi, n, nb, world):
    """Same step through the host-buffer entry points: every save uploads x from pinned host memory and
    downloads ids, offsets and payload; the recovery uploads and downloads the lost shard."""
    import torch

    hx = torch.empty(n, dtype=torch.float32).pin_memory()
    hx.copy_(x0)
    h_payload = torch.empty(n, dtype=torch.float32).pin_memory()
    h_sel = torch.empty(nb, dtype=torch.int32).pin_memory()
    h_poff = torch.empty(nb + 1, dtype=torch.int64).pin_memory()
    steps = 2
    t_save = t_all = 0.0
    h2d = d2h = 0
    for it in range(steps + 1):
        torch.cuda.synchronize()
        s0 = time.perf_counter()
        ts = 0.0
        h2d = d2h = 0
        for r in R_SWEEP:
            ck.load(z0)  # untimed reset
            torch.cuda.synchronize()
            a = time.perf_counter()
            info = api.scar_ckpt_priority_save_host(ck.ctx, hx, r, h_payload, h_sel, h_poff)
            ts += time.perf_counter() - a
            h2d += n * ELEM
            d2h += int(info.payload_elems) * ELEM + int(info.k) * 4 + (int(info.k) + 1) * 8 + 24
        api.scar_recover_partial_host(ck.ctx, hx, lost_shards)
        h2d += (shard_hi - shard_lo) * ELEM + 8
        d2h += (shard_hi - shard_lo) * ELEM + 32
        torch.cuda.synchronize()
        if it > 0:  # first pass is a warm-up
            t_save += ts
            t_all += time.perf_counter() - s0
        hx[shard_lo:shard_hi].copy_(x0[shard_lo:shard_hi])
    return {"value": world * len(R_SWEEP) * 2 * n * ELEM * steps / t_save / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * t_all / steps,
            "note": "host-buffer C-ABI calls, pinned host memory, copies inside the timed region"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--n-elems", type=int, default=N_ELEMS, help="elements of the parameter vector (default 2**30)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
