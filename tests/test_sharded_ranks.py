"""Bookkeeping of the multi-GPU form of a save on CPU: gloo, world size 2, rendezvous on 127.0.0.1.

Every rank owns a contiguous range of the blocks, scores its own slice (here with the oracle, since there is no
GPU), the score slices are gathered with the library's own gather routine, every rank selects over the gathered
scores and keeps the ids it owns.  The union over ranks must be what the oracle saves on the whole buffer."""

import os
import socket
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload():
    sys.path.insert(0, ROOT)
    from workloads import block_offsets, make_workload

    w = make_workload("mlr", rows=7, cols=10_000)  # 7 rows of 10 blocks (9 x 1024 + 784): 70 blocks, uneven split
    return w, block_offsets(w.geom)


def _worker(rank, world, port, k, q):
    import torch
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import oracle
    from paper_1810_07354_b200.sharded import gather_scores, rank_block_range

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w, boff = _workload()
    nb = boff.size - 1
    lo, hi = rank_block_range(nb, world, rank)
    e0, e1 = int(boff[lo]), int(boff[hi])
    x, z = w.x[e0:e1].copy(), w.z[e0:e1].copy()  # this rank's slice of the parameters
    local_boff = (boff[lo: hi + 1] - boff[lo]).astype(np.uint64)
    local_scores = oracle.block_scores(x, z, local_boff)  # step 1 on the rank's own partition
    scores = gather_scores(torch.from_numpy(local_scores), nb, world, rank).numpy()  # step 2
    sel_global, _ = oracle.select_top_k(np.ascontiguousarray(scores), k)  # step 3, the same on every rank
    mine = sel_global[(sel_global >= lo) & (sel_global < hi)]
    local_sel = (mine - lo).astype(np.uint32)
    payload, poff = oracle.pack(x, local_boff, local_sel)  # step 4 on the rank's own blocks
    oracle.update(z, x, local_boff, local_sel)
    q.put((rank, lo, hi, scores.tobytes(), mine.tolist(), payload.tobytes(), poff.tolist(), z.tobytes()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_together_save_what_one_context_over_the_whole_buffer_saves():
    import torch.multiprocessing as mp

    sys.path.insert(0, ROOT)
    import oracle
    from paper_1810_07354_b200.sharded import rank_block_range

    w, boff = _workload()
    nb = boff.size - 1
    k = 23
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, k, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    whole = oracle.priority_save(w.x, w.z, boff, k=k)
    (r0, lo0, hi0, s0, m0, p0, o0, z0), (r1, lo1, hi1, s1, m1, p1, o1, z1) = out
    assert (lo0, hi0, lo1, hi1) == (0, 35, 35, 70) == (*rank_block_range(nb, 2, 0), *rank_block_range(nb, 2, 1))
    assert s0 == s1 == whole.scores.tobytes(), "gathered scores differ from the scores of the whole buffer"
    assert m0 + m1 == whole.sel.tolist(), "the ranks' ids together are not the global selection"
    assert len(m0) + len(m1) == k
    assert p0 + p1 == whole.payload.tobytes(), "payloads in rank order are the payload of the whole buffer"
    assert o0[-1] + o1[-1] == int(whole.poff[-1]) and o0 == whole.poff[: len(m0) + 1].tolist()
    assert z0 + z1 == whole.z_after.tobytes()


def test_rank_ranges_partition_the_blocks():
    sys.path.insert(0, ROOT)
    from paper_1810_07354_b200.sharded import rank_block_range

    for nb in (0, 1, 7, 70, 98_000, 262_144):
        for world in (1, 2, 3, 8):
            r = [rank_block_range(nb, world, i) for i in range(world)]
            assert r[0][0] == 0 and r[-1][1] == nb
            assert all(a[1] == b[0] for a, b in zip(r, r[1:]))
            assert max(b - a for a, b in r) - min(b - a for a, b in r) <= 1
