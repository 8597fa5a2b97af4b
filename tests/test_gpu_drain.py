"""Asynchronous drain of a save's output to pinned host memory (Section 4.3: output to storage happens in the
background while training resumes): what arrives on the host is byte for byte what the oracle packs."""

import numpy as np
import pytest

import oracle
from workloads import block_offsets, make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def check_drained(view, ora):
    assert int(view["info"].k) == ora.k and int(view["info"].payload_elems) == ora.payload.size
    np.testing.assert_array_equal(view["sel"], ora.sel)
    np.testing.assert_array_equal(view["poff"], ora.poff)
    assert parity.same_bits(view["payload"], ora.payload)


@pytest.mark.parametrize("name,kw", [("tiny", dict(n_elems=1 << 18)), ("mlr", dict(rows=8)), ("lda", dict(vocab=2000))])
def test_pipelined_saves_arrive_intact(name, kw):
    """Saves keep coming while the previous one is still being copied out; x changes right after every save."""
    w = make_workload(name, **kw)
    boff = block_offsets(w.geom)
    nb = boff.size - 1
    r = rng(31)
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    k = nb // 5
    max_len = int(np.diff(boff.astype(np.int64)).max())
    ck.drain_init(k, k * max_len)
    hx, hz = w.x.copy(), w.z.copy()
    pending = None  # (ticket, oracle result) of the save that is draining
    for step in range(7):
        strategy = ("priority", "round", "random")[step % 3]
        if strategy == "priority":
            ora = oracle.priority_save(hx, hz, boff, k=k)
            info = ck.priority_save_k(k)
            parity.check_save(ck, info, hx, hz, boff, ora)
        elif strategy == "round":
            cur = ck.round_cursor()
            sel, _ = oracle.select_round(nb, k, cur)
            ora = oracle.save_selected(hx, hz, boff, sel)
            ck.save_round(k, sync=False)
        else:
            pri = r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32)
            ora = oracle.save_selected(hx, hz, boff, oracle.select_random(pri, k))
            ck.save_random(k, parity.to_dev(pri.view(np.int32)), sync=False)
        hz = ora.z_after
        ticket = ck.drain_enqueue()
        # training goes on at once: x changes while the payload of the save above is still on its way out
        if hx.dtype == np.float32:
            hx = (hx + r.standard_normal(hx.size).astype(np.float32) * 0.01).astype(np.float32)
        else:
            hx = np.maximum(hx + r.integers(-2, 3, size=hx.size), 0).astype(np.int32)
        xd.copy_(torch.from_numpy(hx))
        if pending is not None:
            view = ck.drain_wait(pending[0])
            check_drained(view, pending[1])
            assert ck.drain_done(pending[0])
            ck.drain_release(pending[0])
        pending = (ticket, ora)
    view = ck.drain_wait(pending[0])
    check_drained(view, pending[1])
    # the device views still show the most recent save
    dv = ck.views(int(view["info"].k), int(view["info"].payload_elems))
    assert parity.same_bits(dv["payload"].cpu().numpy(), pending[1].payload)
    ck.drain_release(pending[0])
    assert parity.same_bits(ck.views()["z"].cpu().numpy(), hz)
    ck.close()


def test_drain_state_and_capacity_errors():
    w = make_workload("tiny", n_elems=1 << 16)
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    nb, blk = ck.n_blocks, w.geom.block_elems
    with pytest.raises(api.ScarError) as e:
        ck.drain_enqueue()  # not in drain mode
    assert e.value.code == -5
    with pytest.raises(api.ScarError):
        ck.drain_init(nb + 1, 16)
    ck.drain_init(32, 32 * blk)
    with pytest.raises(api.ScarError) as e:
        ck.drain_init(32, 32 * blk)  # once per context
    assert e.value.code == -5
    with pytest.raises(api.ScarError) as e:
        ck.drain_enqueue()  # nothing saved yet
    assert e.value.code == -5
    with pytest.raises(api.ScarError) as e:
        ck.priority_save_k(33)  # more blocks than a slot holds
    assert e.value.code == -7
    ck.priority_save_k(32)
    t1 = ck.drain_enqueue()
    with pytest.raises(api.ScarError) as e:
        ck.drain_enqueue()  # the save was already handed over
    assert e.value.code == -5
    ck.priority_save_k(16)  # second slot
    t2 = ck.drain_enqueue()
    assert t2 != t1
    with pytest.raises(api.ScarError) as e:
        ck.priority_save_k(8)  # both slots are out
    assert e.value.code == -5
    v1 = ck.drain_wait(t1)
    assert int(v1["info"].k) == 32 and v1["payload"].size == 32 * blk
    with pytest.raises(api.ScarError) as e:
        ck.save_round(8)  # waited but not released: the host still owns the buffers
    assert e.value.code == -5
    ck.drain_release(t1)
    ck.priority_save_k(8)
    with pytest.raises(api.ScarError):
        ck.drain_wait(t1)  # released tickets are gone
    ck.drain_release(t2)  # release without wait: waits for the copy itself
    t3 = ck.drain_enqueue()
    assert int(ck.drain_wait(t3)["info"].k) == 8
    ck.drain_release(t3)
    ck.save_round(0)
    t3 = ck.drain_enqueue()
    v3 = ck.drain_wait(t3)
    assert int(v3["info"].k) == 0 and v3["payload"].size == 0 and v3["poff"].tolist() == [0]
    ck.drain_release(t3)
    ck.close()


def test_drain_overlaps_the_next_save():
    """The drain runs on its own stream: while a large payload is on its way to the host the context's stream is
    free to take the next save, which finishes first."""
    n, blk = 1 << 26, 4096
    nb = n // blk
    g = torch.Generator(device="cuda").manual_seed(1)
    z0 = torch.randn(n, device="cuda", generator=g)
    x = z0 + torch.randn(n, device="cuda", generator=g) * 0.01
    ck = api.ScarCheckpoint(x, n_shards=8, block_elems=blk)
    ck.load(z0)
    k = nb // 2
    ck.drain_init(k, k * blk)
    ck.priority_save_k(k)  # 128 MiB payload: a few milliseconds over PCIe
    t1 = ck.drain_enqueue()
    ck.priority_save_k(64, sync=False)  # the next save: kernels only (well under a millisecond), on the context's stream
    ev = torch.cuda.Event()
    ev.record()
    ev.synchronize()
    # The second save has finished.  Had it queued behind the copy, the copy would have finished first; it is
    # still running (128 MiB need at least 2 ms on any PCIe link, the save 0.2 ms).
    assert not ck.drain_done(t1), "the next save waited for the drain of the previous payload"
    v1 = ck.drain_wait(t1)
    info, _ = api.scar_ckpt_last_info(ck.ctx, True, False)
    assert int(v1["info"].k) == k and int(info.k) == 64
    # sampled blocks of the drained payload equal x
    sel = v1["sel"]
    xs = x.cpu().numpy()
    for j in rng(2).integers(0, k, size=32):
        b = int(sel[j])
        assert parity.same_bits(v1["payload"][j * blk:(j + 1) * blk], xs[b * blk:(b + 1) * blk])
    ck.drain_release(t1)
    ck.close()
