"""The multi-GPU form of a save on one GPU: contexts over the parts of one buffer plus the exchange of their score
arrays (a concatenation here, an all-gather between GPUs) must save exactly what one context over the whole
buffer saves, which in turn is what the oracle saves."""

import numpy as np
import pytest

import oracle
from workloads import block_offsets, make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402
from paper_1810_07354_b200.sharded import ShardedCheckpoint, rank_block_range  # noqa: E402


def run_sharded(w, boff, world, k):
    """Saves k blocks of the whole buffer through `world` contexts; returns per-rank results and the pieces."""
    nb = boff.size - 1
    parts = []
    for rank in range(world):
        lo, hi = rank_block_range(nb, world, rank)
        e0, e1 = int(boff[lo]), int(boff[hi])
        xd = parity.to_dev(w.x[e0:e1])
        local_boff = (boff[lo: hi + 1] - boff[lo]).astype(np.uint64)
        ck = api.ScarCheckpoint(xd, n_shards=1, block_offsets=local_boff)
        ck.load(parity.to_dev(w.z[e0:e1]))
        ck.block_scores()  # checkpoint step 1 on every part
        parts.append((ck, xd, lo, hi, e0, e1))
    torch.cuda.synchronize()
    scores = torch.cat([p[0].views()["scores"] for p in parts])  # step 2: what an all-gather leaves on every rank
    out = []
    for ck, xd, lo, hi, e0, e1 in parts:
        info = ck.priority_save_sharded(scores, nb, lo, k)  # steps 3 and 4
        got = parity.fetch_save(ck, info)
        out.append((info, got, lo, e0, e1))
    return parts, out


@pytest.mark.parametrize("name,kw,world,ks", [
    ("tiny", dict(n_elems=1 << 18), 2, (0, 1, 256, 1023, 1024)),
    ("mlr", dict(rows=30, cols=10_000), 3, (57, 150)),  # 300 blocks with short row tails, uneven thirds
    ("lda", dict(vocab=5_000, topics=200), 2, (1000,)),  # integer scores: bit-exact by construction
])
def test_parts_of_one_buffer_save_what_the_whole_buffer_saves(name, kw, world, ks):
    w = make_workload(name, **kw)
    boff = block_offsets(w.geom)
    nb = boff.size - 1
    for k in ks:
        ora = oracle.priority_save(w.x, w.z, boff, k=k)
        # one context over the whole buffer
        xd = parity.to_dev(w.x)
        whole = parity.make_ctx(xd, w.z, geom=w.geom)
        got_whole = parity.check_save(whole, whole.priority_save_k(k), w.x, w.z, boff, ora)
        whole.close()
        parts, out = run_sharded(w, boff, world, k)
        sel = np.concatenate([g["sel"].astype(np.int64) + lo for _, g, lo, _, _ in out]).astype(np.uint32)
        payload = np.concatenate([g["payload"] for _, g, _, _, _ in out])
        z_after = np.concatenate([g["z"] for _, g, _, _, _ in out])
        assert sum(int(i.k) for i, _, _, _, _ in out) == k
        assert np.array_equal(sel, got_whole["sel"]), "the parts' ids together are not the single-context selection"
        assert parity.same_bits(payload, got_whole["payload"]) and parity.same_bits(z_after, got_whole["z"])
        for info, g, lo, e0, e1 in out:  # offsets are local to each rank's payload
            lens = np.diff(boff.astype(np.int64))[g["sel"].astype(np.int64) + lo]
            assert g["poff"].tolist() == np.concatenate([[0], np.cumsum(lens)]).tolist()
            assert int(info.nonfinite_blocks) == ora.nonfinite_blocks
        for ck, *_ in parts:
            ck.close()


def test_sharded_wrapper_on_a_single_rank_and_recovery_stays_local():
    """World size 1 through the wrapper class (the gather is the identity), then a recovery on the same context:
    nothing about recovery needs the other ranks."""
    w = make_workload("tiny", n_elems=1 << 16)
    boff = block_offsets(w.geom)
    xd = parity.to_dev(w.x)
    sc = ShardedCheckpoint(xd, w.n_blocks, 1, 0, n_shards=8, block_elems=w.geom.block_elems)
    sc.ck.load(parity.to_dev(w.z))
    ora = oracle.priority_save(w.x, w.z, boff, r=0.25)
    got = parity.check_save(sc.ck, sc.priority_save(r=0.25), w.x, w.z, boff, ora)
    z_now = parity.next_checkpoint(w.z, w.x, boff, got, ora)
    lost = oracle.expand_shards(w.n_blocks, w.lost_shards)
    want, x_after = oracle.recover_partial(w.x, z_now, boff, lost)
    parity.check_norm(sc.ck.recover_partial(w.lost_shards), want, True)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    with pytest.raises(ValueError):
        ShardedCheckpoint(parity.to_dev(w.x), w.n_blocks + 5, 1, 0, block_elems=w.geom.block_elems)
    sc.close()


def test_sharded_save_argument_errors():
    w = make_workload("tiny", n_elems=1 << 12)
    xd = parity.to_dev(w.x)
    ck = api.ScarCheckpoint(xd, n_shards=1, block_elems=w.geom.block_elems)
    nb = ck.n_blocks
    lib = api.load_library()
    info = api.scar_save_info()
    import ctypes as C

    scores = ck.views()["scores"]
    assert lib.scar_ckpt_priority_save_sharded(ck.ctx, scores.data_ptr(), nb, 1, 1, C.byref(info)) == -1  # range past the end
    assert lib.scar_ckpt_priority_save_sharded(ck.ctx, scores.data_ptr(), nb, 0, nb + 1, C.byref(info)) == -1
    assert lib.scar_ckpt_priority_save_sharded(ck.ctx, None, nb, 0, 1, C.byref(info)) == -1
    assert lib.scar_ckpt_priority_save_sharded(ck.ctx, scores.data_ptr(), nb, 0, 1, None) == -1
    ck.close()
