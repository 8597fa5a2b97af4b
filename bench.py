#!/usr/bin/env python
"""Benchmark of the SCAR checkpoint-and-recover pass.

Default workload: the CNN-scale parameter set, 2**30 float32 elements in 4096-element blocks.  One
step = the whole hot path over one synthetic parameter set: a prioritized save at every r of the set's
sweep (CNN: 0.01, 0.1, 0.5, 1.0; the running checkpoint is put back to its pristine state and L2 is
flushed before each, outside the timed intervals), the read-only full-recovery perturbation norm, and
a partial recovery of the set's lost shards or blocks.  Every timed call is bracketed by CUDA events on
the stream the library launches on; a step's time is the sum of its timed calls.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its own GPU:
the pass over one device's parameters needs no exchange, so there is no collective on the data path;
the reported value is the sum over ranks divided by the slowest rank's time.

``--impl reference`` times the plain CPU oracle (``oracle/``) on the host cores over a bounded sample
of the same parameter set, with the same metric.  ``--workload`` selects one of the other synthetic
sets (tiny, mlr, mf, lda) for the same measurement.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N_ELEMS = 1 << 30
BLOCK = 4096
ELEM = 4
METRIC = "prioritized-checkpoint GB/s scanned"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0

DESCRIPTIONS = {
    "cnn": "cnn-scale fp32 vector, block 4096, r sweep 0.01/0.1/0.5/1.0 + full norm + recovery of 1 of 8 shards",
    "mlr": "mlr-shaped fp32 1000x100000, blocks of 1024 within rows, r 0.05/0.25 + full norm + recovery of 1 of 8 "
           "row shards",
    "mf": "mf-shaped fp32 factors (480000+18000)x100, one 100-float row per block, r 0.1 + full norm + recovery of "
          "a random 25% of L rows",
    "lda": "lda-shaped int32 100000x1000 count table, one row per block, integer l1, r 0.2 + full norm + recovery "
           "of 2 of 8 shards",
    "tiny": "tiny fp32 vector 2**20, block 256, r 0.25 + full norm + recovery of 4 of 8 shards (L2-resident: "
            "latency-bound, not an HBM measurement)",
}


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def recorded_traffic(n_elems: int, kernel: str = "k_block_scores"):
    """DRAM bytes per launch of the dominant kernel from the last ncu capture, scaled to n_elems; None when
    there is no capture or the kernel sources changed after it was taken."""
    import hashlib

    pkg = os.path.join(ROOT, "paper_1810_07354_b200")
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            rec = json.load(f)[kernel]
        h = hashlib.sha256()
        for name in ("geom.cuh", "sel_state.cuh", "block_pass.cuh"):
            with open(os.path.join(pkg, "csrc", name), "rb") as f:
                h.update(f.read())
        if h.hexdigest() != rec["src_sha256"]:
            return None
        return rec["dram_bytes_per_launch"] * (n_elems / rec["n_elems"])
    except Exception:
        return None


def save_bytes(n_elems: int, payload_elems: int) -> int:
    """Algorithmic bytes of one save: both streams read once, the selected blocks read again and written twice.
    A full checkpoint (everything selected) needs no second read: the selection is known before the scan."""
    if payload_elems == n_elems:
        return 4 * n_elems * ELEM
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


def oracle_step(x, z, boff, lost_blocks, r_sweep):
    """One step of the hot path on the oracle; returns seconds spent in saves and in total."""
    import oracle

    t_save = 0.0
    t0 = time.perf_counter()
    for r in r_sweep:
        t = time.perf_counter()
        oracle.priority_save(x, z, boff, r=r)
        t_save += time.perf_counter() - t
    oracle.perturbation_norm(x, z, boff, None)
    oracle.recover_partial(x, z, boff, lost_blocks)
    return t_save, time.perf_counter() - t0


def host_workload(name: str, n_elems: int):
    """Host (numpy) form of a workload; only the CNN-scale set takes a size."""
    from workloads import make_workload

    if name == "cnn":
        return make_workload("cnn", n_elems=n_elems, block_elems=BLOCK)
    return make_workload(name)


def lost_block_mask(w):
    import oracle

    return w.lost_blocks if w.lost_blocks is not None else oracle.expand_shards(w.n_blocks, w.lost_shards)


def run_reference(args):
    """The oracle as it stands, single-threaded, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from workloads import block_offsets

    # One oracle step over 2**26 CNN-scale elements takes 2-5 s; shrink the sample so that warm-up plus
    # timed steps stay within a couple of minutes.  The other sets (<= 1e8 elements) are used whole.
    n = 1 << 26
    while n > (1 << 22) and 5.0 * (n / (1 << 26)) * (args.steps + args.warmup) > 120.0:
        n >>= 1
    n = max(BLOCK, min(n, args.n_elems))
    w = host_workload(args.workload, n)
    n = w.x.size
    full = N_ELEMS if args.workload == "cnn" else n
    boff = block_offsets(w.geom)
    lost = lost_block_mask(w)
    for _ in range(args.warmup):
        oracle_step(w.x, w.z, boff, lost, w.r_values)
    t_save = t_all = 0.0
    for _ in range(args.steps):
        a, b = oracle_step(w.x, w.z, boff, lost, w.r_values)
        t_save += a
        t_all += b
    value = len(w.r_values) * 2 * n * ELEM * args.steps / t_save / 1e9
    sample = f"{n} of {full} elements ({w.n_blocks} blocks), numpy-generated with the same recipe"
    nproc, model = host_cpu()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64" if w.dtype == "f32" else "int64", "data": "synthetic",
        "config": {"workload": DESCRIPTIONS[args.workload] + (f" [sample: {n} of {full} elements]" if n != full else ""),
                   "n_elems": n, "sample_of": full},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample, "nproc": nproc,
                         "cpu_model": model},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def host_cpu():
    """(logical cores, model string) of the host."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return os.cpu_count() or 1, model


def time_oracle_steps(x, z, boff, lost_blocks, r_sweep, budget_s=5.0, max_reps=50):
    """Repeats the oracle step until a few seconds of saves have been timed; (GB/s scanned, reps, seconds)."""
    reps, t_save = 0, 0.0
    while reps < 1 or (t_save < budget_s and reps < max_reps):
        t_save += oracle_step(x, z, boff, lost_blocks, r_sweep)[0]
        reps += 1
    return reps * len(r_sweep) * 2 * x.size * ELEM / t_save / 1e9, reps, t_save


def cpu_baseline(x_dev, z_dev, geom, lost_blocks, r_sweep):
    """Times the oracle on the device-resident workload (copied to the host): as it stands on one thread, and the
    same source built with OpenMP (loops over blocks in parallel, the selection still the serial sort) on all
    cores.  The headline `value` is the single-thread leg, the oracle exactly as the parity tests use it."""
    import oracle
    from workloads import block_offsets

    x = x_dev.cpu().numpy()
    z = z_dev.cpu().numpy()
    boff = block_offsets(geom)
    nproc, model = host_cpu()
    what = f"all {x.size} elements ({geom.n_blocks} blocks) of the same buffers"
    v1, reps1, t1 = time_oracle_steps(x, z, boff, lost_blocks, r_sweep)
    legs = {"single_thread": {"value": v1, "unit": UNIT, "cores": 1, "sample": f"{reps1} step(s) on {what}, {t1:.1f} s in saves"}}
    try:
        threads = oracle.use_openmp(True)
        oracle_step(x, z, boff, lost_blocks, r_sweep)  # first touch by the thread pool, untimed
        vn, repsn, tn = time_oracle_steps(x, z, boff, lost_blocks, r_sweep)
        legs["all_cores"] = {"value": vn, "unit": UNIT, "cores": threads,
                             "sample": f"{repsn} step(s) on {what}, {tn:.1f} s in saves; OpenMP build of the same "
                                       "source, selection serial"}
    except Exception as e:  # no OpenMP runtime on the host: say so, keep the single-thread leg
        legs["all_cores"] = {"unavailable": str(e)[:200]}
    finally:
        oracle.use_openmp(False)
    return {"value": v1, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": legs["single_thread"]["sample"],
            "nproc": nproc, "cpu_model": model, **legs}


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


def device_workload(name, n_elems, rank, dev):
    """(geom, z0, x0, r_sweep, lost_shards, lost_blocks_host) with z0 / x0 on the device."""
    import torch

    if name == "cnn":
        from workloads.configs import make_cnn_device

        geom, z0, x0, lost_shards = make_cnn_device(n_elems, BLOCK, seed=4 + rank, device=dev)
        return geom, z0, x0, (0.01, 0.1, 0.5, 1.0), lost_shards, None
    from workloads import make_workload

    w = make_workload(name)
    return (w.geom, torch.from_numpy(w.z).to(dev), torch.from_numpy(w.x).to(dev), w.r_values, w.lost_shards,
            w.lost_blocks)


class L2Flush:
    """Empties the L2 cache of everything a timed call could reuse: writes a 256 MiB buffer (twice the 126 MB
    L2), then reads another 256 MiB one.  The read pass matters for the small parameter sets: a write-only flush
    leaves the cache full of the flush buffer's dirty lines, and the next call then pays for writing them back
    (up to 126 MB of foreign DRAM traffic inside a call that itself moves 150 to 900 MB); after the read pass the
    cache holds clean lines that are dropped for free.  Always outside the timed intervals."""

    def __init__(self, dev):
        import torch

        self.w = torch.empty(64 << 20, dtype=torch.float32, device=dev)
        self.r = torch.zeros(64 << 20, dtype=torch.float32, device=dev)
        self.sink = None

    def zero_(self):
        self.w.zero_()
        self.sink = self.r.sum()


class Measured:
    """Raw results of the timed steps of one workload on this rank."""


def measure_workload(api, name, n_elems, rank, dev, steps, warmup, barrier):
    """W warm-up steps, then `steps` timed steps of the whole hot path over one synthetic parameter set, each
    call bracketed by CUDA events on the stream the library launches on; then the per-phase durations through
    the library's own events.  Returns a Measured holding the context and the buffers (the caller frees them)."""
    import torch

    m = Measured()
    m.name = name
    geom, z0, x0, r_sweep, lost_shards, lost_blocks = device_workload(name, n_elems, rank, dev)
    m.geom, m.z0, m.x0, m.r_sweep, m.lost_shards, m.lost_blocks = geom, z0, x0, r_sweep, lost_shards, lost_blocks
    m.n = x0.numel()
    m.x = x0.clone()
    m.ck = ck = api.ScarCheckpoint(m.x, n_shards=geom.n_shards, row_elems=geom.row_elems, block_elems=geom.block_elems)
    ctx = ck.ctx
    m.nb = ck.n_blocks
    d_lost = torch.from_numpy(lost_blocks).to(dev) if lost_blocks is not None else None

    def recover(sync=False):
        if d_lost is not None:
            return ck.recover_partial_blocks(d_lost, sync=sync)
        return ck.recover_partial(lost_shards, sync=sync)

    m.z_lib = z_lib = ck.views()["z"]  # the library's running checkpoint, aliased (no copy)
    m.flush = flush = L2Flush(dev)

    def reset_checkpoint():
        """Pristine running checkpoint, then an L2 flush; plain torch copies, outside every timed interval."""
        z_lib.copy_(z0)
        flush.zero_()

    def reset_live():
        m.x.copy_(x0)
        flush.zero_()

    m.lost_elems = int(recover(sync=True).lost_elems)
    reset_live()

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def one_step(rec):
        """Runs one step; appends (kind, start_event, end_event) triples to rec."""
        for r in r_sweep:
            reset_checkpoint()
            a, b = ev(), ev()
            a.record()
            ck.priority_save(r, sync=False)
            b.record()
            rec.append((("save", r), a, b))
        reset_checkpoint()
        a, b = ev(), ev()
        a.record()
        ck.perturbation_norm(None, sync=False)
        b.record()
        rec.append((("norm", None), a, b))
        flush.zero_()
        a, b = ev(), ev()
        a.record()
        recover()
        b.record()
        rec.append((("recover", None), a, b))
        reset_live()  # put the live parameters back (not timed)

    for _ in range(warmup):
        one_step([])
    barrier()

    # payload sizes per r (data dependent but fixed for this workload)
    m.payload_elems = {}
    for r in r_sweep:
        reset_checkpoint()
        m.payload_elems[r] = int(ck.priority_save(r).payload_elems)
    barrier()

    # ---- timed region: K steps, device-timed
    launches0 = api.scar_ckpt_launch_count(ctx)
    rec = []
    barrier()
    m.w0 = time.time()
    for _ in range(steps):
        one_step(rec)
    barrier()
    m.w1 = time.time()
    m.launches = api.scar_ckpt_launch_count(ctx) - launches0
    m.t = {}
    for (kind, r), a, b in rec:
        m.t.setdefault((kind, r), []).append(a.elapsed_time(b))

    # ---- phases (and with them the dominant kernel, block scores) timed live through the library's own
    # stream events
    api.scar_ckpt_profile(ctx, True)
    m.phase = {r: [] for r in r_sweep}
    m.rec_phase = []
    for _ in range(min(steps, 10)):
        for r in r_sweep:
            reset_checkpoint()
            ck.priority_save(r, sync=False)
            m.phase[r].append(api.scar_ckpt_profile_read(ctx))
        flush.zero_()
        recover()
        m.rec_phase.append(api.scar_ckpt_profile_read(ctx))
        reset_live()
    api.scar_ckpt_profile(ctx, False)
    # the scoring kernel runs on its own in every save that is not a full checkpoint (those fuse it with the pack)
    partial = [r for r in r_sweep if m.payload_elems[r] < m.n] or list(r_sweep)
    m.score_ms = float(np.mean([p[0] for r in partial for p in m.phase[r]]))
    return m


def event_floor(dev, reps=50):
    """What a pair of CUDA events reads around a kernel that does nothing: a one-element fill launched behind a
    kernel that is still running, as every timed phase is.  The phase times of the small parameter sets (the
    selection above all) contain this much that is not the kernel."""
    import torch

    one = torch.zeros(1, device=dev)
    busy = torch.zeros(1 << 24, device=dev)
    ts = []
    for _ in range(reps + 5):
        busy.add_(1.0)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        one.zero_()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    ts = ts[5:]
    return {"ms": float(np.median(ts)), "ms_min": float(np.min(ts)),
            "what": "a one-element fill between two events, behind a running kernel"}


def graph_saves(api, name, dev, reps=20):
    """The saves of one small parameter set recorded once in a CUDA graph and replayed: what a save costs when
    its three launches are issued by the device instead of one by one from the host (the sets whose kernels
    are shorter than a launch call).  Same events, same L2 flush, same reset of the running checkpoint as the
    eager measurement."""
    import torch

    geom, z0, x0, r_sweep, _, _ = device_workload(name, 0, 0, dev)
    s = torch.cuda.Stream()
    x = x0.clone()
    torch.cuda.synchronize()
    ck = api.ScarCheckpoint(x, n_shards=geom.n_shards, row_elems=geom.row_elems, block_elems=geom.block_elems, stream=s)
    z_lib = ck.views()["z"]
    flush = L2Flush(dev)
    out = {}
    with torch.cuda.stream(s):
        for r in r_sweep:
            ck.priority_save(r, sync=False)  # every kernel has run once before anything is recorded
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                ck.priority_save(r, sync=False)
            ts = []
            for _ in range(reps + 3):
                z_lib.copy_(z0)
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s)
                g.replay()
                b.record(s)
                b.synchronize()
                ts.append(a.elapsed_time(b))
            out[str(r)] = {"save_ms": float(np.median(ts[3:])), "save_ms_min": float(np.min(ts[3:]))}
            del g
    s.synchronize()
    ck.close()
    return out


def summarise(m, peak):
    """Per-r save figures, norm and recovery figures of one measured workload."""
    scanned = 2 * m.n * ELEM
    per_r = {}
    for r in m.r_sweep:
        ms = float(np.median(m.t[("save", r)]))
        by = save_bytes(m.n, m.payload_elems[r])
        ph = np.median(np.array(m.phase[r]), axis=0)
        per_r[str(r)] = {"save_ms": ms, "save_ms_min": float(np.min(m.t[("save", r)])), "scanned_gbs": scanned / ms / 1e6,
                         "algorithmic_gbs": by / ms / 1e6, "frac_of_measured_peak": by / ms / 1e6 / peak,
                         "frac_of_8tbs": by / ms / 1e6 / 8000.0, "blocks_per_s": m.nb / (ms * 1e-3),
                         "payload_elems": m.payload_elems[r],
                         "phase_ms": {"scores": float(ph[0]), "select": float(ph[1]), "pack": float(ph[2])}}
    norm_ms = float(np.median(m.t[("norm", None)]))
    rec_ms = float(np.median(m.t[("recover", None)]))
    rph = np.median(np.array(m.rec_phase), axis=0)
    rec_gbs = 3 * m.lost_elems * ELEM / rec_ms / 1e6
    return {
        "per_r": per_r,
        "perturbation_norm": {"ms": norm_ms, "gbs": scanned / norm_ms / 1e6, "frac_of_measured_peak": scanned / norm_ms / 1e6 / peak},
        "partial_recovery": {"ms": rec_ms, "gbs": rec_gbs, "frac_of_measured_peak": rec_gbs / peak,
                             "lost_elems": m.lost_elems, "phase_ms": {"restore_and_norm": float(rph[3])}},
        "block_scores": {"ms": m.score_ms, "gbs": scanned / m.score_ms / 1e6, "frac_of_measured_peak": scanned / m.score_ms / 1e6 / peak},
    }


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_1810_07354_b200 import api

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

    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid)) if rank == 0 else None
    m = measure_workload(api, args.workload, args.n_elems, rank, dev, args.steps, args.warmup, barrier)
    clocks = sampler.stop(m.w0, m.w1) if sampler else None
    n, nb, r_sweep = m.n, m.nb, m.r_sweep

    tot_ms = sum(sum(v) for v in m.t.values())
    save_ms = sum(sum(v) for (kind, _), v in m.t.items() if kind == "save")
    tot_ms, save_ms = max_over_ranks([tot_ms, save_ms], dev, world)

    if rank != 0:
        barrier()
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = hbm_peak()
    scanned = 2 * n * ELEM
    value = job_throughput_gbs(world, len(r_sweep) * scanned * args.steps, save_ms)
    summ = summarise(m, peak)
    achieved = scanned / (m.score_ms * 1e-3) / 1e9
    l2_note = ("inputs larger than L2; " if scanned > (512 << 20) else "inputs NOT larger than L2; ") + \
        "L2 flushed by a 256 MiB write followed by a 256 MiB read after every untimed state reset and before every timed call"

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": tot_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if m.x0.dtype == torch.float32 else "int32", "data": "synthetic",
        "config": {"workload": DESCRIPTIONS[args.workload], "n_elems": n, "n_blocks": nb, "r_sweep": list(r_sweep),
                   "l2": l2_note, "value_is": "sum over the r sweep of 2*N*4 bytes / sum of save times",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "save_ms_per_step": save_ms / args.steps,
        "per_r": summ["per_r"],
        "perturbation_norm": summ["perturbation_norm"],
        "partial_recovery": summ["partial_recovery"],
        "roofline": {"bound": "hbm", "kernel": "k_block_scores", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                     "traffic": recorded_traffic(n) if args.workload == "cnn" else None,
                     "bytes_per_launch": scanned, "ms_per_launch": m.score_ms},
        "gpu_launches": int(m.launches),
        "event_floor": event_floor(dev),
        "clocks": clocks,
        "wall_s_timed_region": m.w1 - m.w0,
    }

    if not args.no_e2e:
        line["e2e"] = run_e2e(api, m.ck, m.x0, m.z_lib, m.z0, r_sweep, m.lost_shards, m.lost_elems, n, nb, world, m.flush)
    if world == 1 and not args.no_cpu_baseline:
        if m.lost_blocks is None:
            from workloads import shard_block_ranges

            lb = np.zeros(nb, dtype=np.uint8)
            for lo, hi in shard_block_ranges(nb, m.geom.n_shards)[np.flatnonzero(m.lost_shards)]:
                lb[lo:hi] = 1
        else:
            lb = m.lost_blocks
        line["cpu_baseline"] = cpu_baseline(m.x0, m.z0, m.geom, lb, r_sweep)
    if world == 1 and not args.no_extras:
        line["extras"] = run_extras(api, m.ck, m.x, m.x0, m.z_lib, m.z0, m.geom, r_sweep, m.flush, dev,
                                    with_bylayer=args.workload == "cnn" and n >= (1 << 28))
    if world == 1 and args.workload == "cnn" and not args.no_configs:
        # The other four parameter sets (far smaller: their steps take a fraction of a millisecond) measured the
        # same way, after the headline's buffers are gone; same keys per set, fewer steps.
        configs = {"cnn": summ}
        m.ck.close()
        del m
        torch.cuda.empty_cache()
        for name in ("tiny", "mlr", "mf", "lda"):
            mm = measure_workload(api, name, 0, rank, dev, min(args.steps, 20), max(args.warmup, 3), barrier)
            configs[name] = dict(summarise(mm, peak), n_elems=mm.n, n_blocks=mm.nb, workload=DESCRIPTIONS[name],
                                 gpu_launches=int(mm.launches))
            mm.ck.close()
            del mm
            torch.cuda.empty_cache()
            configs[name]["graph_replay"] = graph_saves(api, name, dev)
            torch.cuda.empty_cache()
        line["configs"] = configs
    print(json.dumps(line))
    barrier()
    if world > 1:
        dist.destroy_process_group()


def run_sharded(args):
    """The multi-GPU form of the save (Section 4.3 with one GPU per node): the CNN-scale parameter vector is
    split over the ranks by blocks, every rank scores its slice, one all-gather makes all scores known, every
    rank selects the same global fraction and saves the blocks it owns.  Total work is fixed as N grows
    ("scaling": "strong").  A step = one sharded save per r of the sweep + the rank's full norm + a recovery of
    one of its 8 local shards; device-timed per call, maximum over ranks."""
    import torch
    import torch.distributed as dist

    from paper_1810_07354_b200 import api
    from paper_1810_07354_b200.sharded import ShardedCheckpoint, rank_block_range
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

    nb_global = args.n_elems // BLOCK
    lo, hi = rank_block_range(nb_global, world, rank)
    n = (hi - lo) * BLOCK
    _, z0, x0, lost_shards = make_cnn_device(n, BLOCK, seed=4 + rank, device=dev)
    x = x0.clone()
    sc = ShardedCheckpoint(x, nb_global, world, rank, n_shards=8, block_elems=BLOCK)
    z_lib = sc.ck.views()["z"]
    flush = L2Flush(dev)
    r_sweep = (0.01, 0.1, 0.5, 1.0)
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def one_step(rec):
        for r in r_sweep:
            z_lib.copy_(z0)
            flush.zero_()
            barrier()  # the exchange inside the save would otherwise absorb the ranks' skew
            a, b = ev(), ev()
            a.record()
            sc.priority_save(r=r)
            b.record()
            rec.append((("save", r), a, b))
        z_lib.copy_(z0)
        flush.zero_()
        a, b = ev(), ev()
        a.record()
        sc.ck.perturbation_norm(None, sync=False)
        b.record()
        rec.append((("norm", None), a, b))
        flush.zero_()
        a, b = ev(), ev()
        a.record()
        sc.ck.recover_partial(lost_shards, sync=False)
        b.record()
        rec.append((("recover", None), a, b))
        x.copy_(x0)

    for _ in range(args.warmup):
        one_step([])
    barrier()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid)) if rank == 0 else None
    launches0 = api.scar_ckpt_launch_count(sc.ck.ctx)
    rec = []
    barrier()
    w0 = time.time()
    for _ in range(args.steps):
        one_step(rec)
    barrier()
    w1 = time.time()
    launches = api.scar_ckpt_launch_count(sc.ck.ctx) - launches0
    clocks = sampler.stop(w0, w1) if sampler else None
    t = {}
    for key, a, b in rec:
        t.setdefault(key, []).append(a.elapsed_time(b))
    keys = sorted(t, key=str)
    sums = max_over_ranks([sum(t[k]) for k in keys], dev, world)
    tot = dict(zip(keys, sums))
    if rank == 0:
        save_ms = sum(v for (kind, _), v in tot.items() if kind == "save")
        tot_ms = sum(tot.values())
        scanned = 2 * nb_global * BLOCK * ELEM
        peak, peak_kind = hbm_peak()
        line = {
            "metric": METRIC, "value": len(r_sweep) * scanned * args.steps / (save_ms * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_ms / args.steps,
            "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": DESCRIPTIONS["cnn"] + " [blocks split over the ranks, global top-r]",
                       "n_elems": nb_global * BLOCK, "n_blocks": nb_global, "r_sweep": list(r_sweep),
                       "parallelism": f"blocks sharded x{world}, one all-gather of the scores per save",
                       "l2": "per-rank inputs larger than L2 up to 8 ranks; L2 flushed before every timed call"},
            "per_r": {str(r): {"save_ms": tot[("save", r)] / args.steps,
                               "scanned_gbs": scanned / (tot[("save", r)] / args.steps) / 1e6} for r in r_sweep},
            "perturbation_norm_ms": tot[("norm", None)] / args.steps,
            "partial_recovery_ms": tot[("recover", None)] / args.steps,
            "roofline": {"bound": "hbm", "kernel": "k_block_scores", "achieved": None, "peak": peak, "unit": "GB/s",
                         "frac": None, "peak_source": f"of {peak_kind}", "traffic": None,
                         "note": "per-kernel figures are those of the single-GPU line; this mode times whole calls"},
            "gpu_launches": int(launches), "clocks": clocks, "wall_s_timed_region": w1 - w0,
        }
        print(json.dumps(line))
    barrier()
    sc.close()
    if world > 1:
        dist.destroy_process_group()


def run_select_stamps(args):
    """Where the selection kernel's time goes: with a diagnostic build of the library
    (``python -m paper_1810_07354_b200._build --select-stamps``) prints, per r of the workload, the microseconds
    between the marked points of the kernel's first CTA (median of 8 saves; SM cycles / the SM clock in MHz).
    Rebuild without the flag afterwards."""
    import torch

    from paper_1810_07354_b200 import api

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    geom, z0, x0, r_sweep, _, _ = device_workload(args.workload, args.n_elems, 0, dev)
    ck = api.ScarCheckpoint(x0.clone(), n_shards=geom.n_shards, row_elems=geom.row_elems, block_elems=geom.block_elems)
    mhz = float(subprocess.run(["nvidia-smi", "-i", "0", "--query-gpu=clocks.max.sm", "--format=csv,noheader,nounits"],
                               capture_output=True, text=True).stdout.split()[0])
    flush = L2Flush(dev)
    out = {"workload": args.workload, "n_blocks": ck.n_blocks, "sm_mhz_assumed": mhz, "per_r": {}}
    for r in r_sweep:
        runs = []
        for _ in range(10):
            ck.load(z0)
            flush.zero_()
            ck.priority_save(r)
            runs.append(api.scar_ckpt_debug_select_stamps(ck.ctx))
        st = np.median(np.array(runs[2:], dtype=np.float64), axis=0)
        us = lambda a, b: round(float(st[b] - st[a]) / mhz, 2)  # noqa: E731
        rec, last = {"keys_loaded": us(0, 1)}, 1
        for p in range(6):
            if st[2 + 4 * p] > st[0]:  # this digit pass ran
                rec[f"pass{p}"] = {"histogram": us(last, 2 + 4 * p), "flush": us(2 + 4 * p, 3 + 4 * p),
                                   "complete_and_resolved": us(3 + 4 * p, 5 + 4 * p)}
                last = 5 + 4 * p
        rec.update(counts=us(last, 26), exchange=us(26, 27), scan=us(27, 28), emit=us(28, 29), total=us(0, 29))
        out["per_r"][str(r)] = rec
    ck.close()
    print(json.dumps(out))


def run_extras(api, ck, x, x0, z_lib, z0, geom, r_sweep, flush, dev, with_bylayer):
    """Measurements beside the headline step, outside its timed region: the two baseline selectors
    (Section 5.4), the asynchronous drain (Section 4.3) and a by-layer layout with very unequal blocks
    (Section 5.1).  Device times from CUDA events / the library's phase events; the drain is wall-clock because
    it ends on the host."""
    import torch

    from workloads import bylayer_offsets

    n, nb = x.numel(), ck.n_blocks
    r = r_sweep[min(1, len(r_sweep) - 1)]
    k = max(1, int(r * nb + 0.5))
    out = {"r": r, "k": k}
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def timed(fn, reps=10):
        ts = []
        for _ in range(reps + 2):
            z_lib.copy_(z0)
            flush.zero_()
            a, b = ev(), ev()
            a.record()
            fn()
            b.record()
            b.synchronize()
            ts.append(a.elapsed_time(b))
        return float(np.median(ts[2:]))

    pri = torch.randint(0, 2**31 - 1, (nb,), device=dev, dtype=torch.int32)
    info = ck.save_round(k)
    pay = int(info.payload_elems)
    for name, fn in (("priority", lambda: ck.priority_save_k(k, sync=False)),
                     ("round", lambda: ck.save_round(k, sync=False)),
                     ("random", lambda: ck.save_random(k, pri, sync=False))):
        ms = timed(fn)
        moved = 3 * pay * ELEM + (2 * n * ELEM if name == "priority" else 0)
        out[name] = {"save_ms": ms, "algorithmic_gbs": moved / ms / 1e6}

    # ---- asynchronous drain: saves keep running on the context's stream while the previous payload goes to
    # pinned host memory on the drain stream
    block_len = geom.block_elems if geom.block_elems else n
    ck.drain_init(k, min(n, k * min(block_len, geom.row_len)))
    dump_ms, tickets, n_saves = [], [], 6
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(n_saves):
        z_lib.copy_(z0)
        a, b = ev(), ev()
        a.record()
        ck.priority_save_k(k, sync=False)
        b.record()
        tickets.append((ck.drain_enqueue(), a, b))
        if len(tickets) >= 2:  # two slots: take the older payload off the host side before the next save
            t_old, a_old, b_old = tickets.pop(0)
            ck.drain_wait(t_old)
            ck.drain_release(t_old)
            dump_ms.append(a_old.elapsed_time(b_old))
    t_old, a_old, b_old = tickets.pop(0)
    view = ck.drain_wait(t_old)
    drained = int(view["info"].payload_elems) * ELEM + int(view["info"].k) * 12 + 40
    ck.drain_release(t_old)
    dump_ms.append(a_old.elapsed_time(b_old))
    wall_ms = 1e3 * (time.perf_counter() - t0) / n_saves
    # one save + drain with nothing else in flight, for the copy rate alone
    z_lib.copy_(z0)
    ck.priority_save_k(k, sync=False)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    t = ck.drain_enqueue()
    ck.drain_wait(t)
    copy_ms = 1e3 * (time.perf_counter() - t1)
    ck.drain_release(t)
    out["drain"] = {"t_dump_ms": float(np.median(dump_ms)), "pipelined_ms_per_save": wall_ms,
                    "drain_alone_ms": copy_ms, "drained_bytes": drained, "drain_gbs": drained / copy_ms / 1e6,
                    "note": "t_dump = score + select + pack + cache refresh on the context's stream while the "
                            "previous payload is copied out; pipelined = wall-clock per save of 6 back-to-back "
                            "save + drain rounds (PCIe-bound)"}

    # ---- by-layer layout: 10 tensors from 12 to 8.2e8 elements, cut into segments by the library
    if with_bylayer:
        boff = bylayer_offsets(scale=16, pad_to=4)
        nl = int(boff[-1])
        g = torch.Generator(device=dev).manual_seed(11)
        zl = torch.randn(nl, device=dev, generator=g) * 5e-2
        xl = zl + torch.randn(nl, device=dev, generator=g) * 1e-3
        cl = api.ScarCheckpoint(xl, n_shards=5, block_offsets=boff)
        api.scar_ckpt_profile(cl.ctx, True)
        rows = []
        for _ in range(5):
            cl.load(zl)
            flush.zero_()
            cl.priority_save_k(5, sync=False)
            ph = api.scar_ckpt_profile_read(cl.ctx)
            pe = int(api.scar_ckpt_last_info(cl.ctx, True, False)[0].payload_elems)
            flush.zero_()
            cl.recover_partial(np.array([0, 0, 1, 0, 0], dtype=np.uint8), sync=False)
            rp = api.scar_ckpt_profile_read(cl.ctx)
            le = int(api.scar_ckpt_last_info(cl.ctx, False, True)[1].lost_elems)
            rows.append((ph[0], ph[1], ph[2], rp[3]))
            xl.copy_(zl + 1e-3)
        m = np.median(np.array(rows[1:]), axis=0)
        out["bylayer"] = {"n_elems": nl, "n_blocks": int(boff.size - 1), "longest_block": int(np.diff(boff.astype(np.int64)).max()),
                          "scores_ms": float(m[0]), "scores_gbs": 2 * nl * ELEM / m[0] / 1e6,
                          "select_ms": float(m[1]), "pack_ms": float(m[2]), "pack_gbs": 3 * pe * ELEM / m[2] / 1e6,
                          "recover_ms": float(m[3]), "recover_gbs": 3 * le * ELEM / m[3] / 1e6, "lost_elems": le}
        cl.close()
    return out


def run_e2e(api, ck, x0, z_lib, z0, r_sweep, lost_shards, lost_elems, n, nb, world, flush):
    """Same step through the host-buffer entry points: every save uploads x from pinned host memory and
    downloads ids, offsets and payload; the recovery (shard-mask workloads) uploads and downloads the lost
    shards.  Wall-clock around the synchronous calls, copies included."""
    import torch

    hx = torch.empty(n, dtype=x0.dtype).pin_memory()
    hx.copy_(x0)
    h_payload = torch.empty(n, dtype=x0.dtype).pin_memory()
    h_sel = torch.empty(nb, dtype=torch.int32).pin_memory()
    h_poff = torch.empty(nb + 1, dtype=torch.int64).pin_memory()
    steps = 2
    t_save = t_all = 0.0
    h2d = d2h = 0
    for it in range(steps + 1):
        torch.cuda.synchronize()
        t_step = 0.0
        ts = 0.0
        h2d = d2h = 0
        for r in r_sweep:
            z_lib.copy_(z0)  # untimed reset
            flush.zero_()
            torch.cuda.synchronize()
            a = time.perf_counter()
            info = api.scar_ckpt_priority_save_host(ck.ctx, hx, r, h_payload, h_sel, h_poff)
            ts += time.perf_counter() - a
            h2d += n * ELEM
            d2h += int(info.payload_elems) * ELEM + int(info.k) * 4 + (int(info.k) + 1) * 8 + 24
        t_step += ts
        if lost_shards is not None:
            a = time.perf_counter()
            api.scar_recover_partial_host(ck.ctx, hx, lost_shards)
            t_step += time.perf_counter() - a
            h2d += lost_elems * ELEM
            d2h += lost_elems * ELEM + 32
            hx.copy_(x0)
        if it > 0:  # first pass is a warm-up
            t_save += ts
            t_all += t_step
    return {"value": world * len(r_sweep) * 2 * n * ELEM * steps / t_save / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * t_all / steps,
            "note": "host-buffer C-ABI calls, pinned host memory, copies inside the timed region"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="cnn", choices=sorted(DESCRIPTIONS))
    ap.add_argument("--n-elems", type=int, default=N_ELEMS,
                    help="elements of the CNN-scale parameter vector (default 2**30)")
    ap.add_argument("--sharded", action="store_true",
                    help="multi-GPU form of the save: the blocks of one parameter vector split over the ranks, "
                         "global top-r through one all-gather of the scores (strong scaling) instead of replicas")
    ap.add_argument("--select-stamps", action="store_true",
                    help="diagnostic builds of the library only: print where the selection kernel spends its time")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="with the default workload: skip the measurement of the four smaller parameter sets")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the measurements beside the headline step (baseline selectors, drain, by-layer layout)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.select_stamps:
        run_select_stamps(args)
    elif args.sharded:
        run_sharded(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
