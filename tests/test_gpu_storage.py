"""The running checkpoint in persistent storage (Sections 4.2 / 4.3): a file that is initialised with x^(0),
receives each partial checkpoint's blocks in the background, and always holds the oracle's running checkpoint;
a fresh context recovers lost parameters from it."""

import os

import numpy as np
import pytest

import oracle
from workloads import block_offsets, make_cnn_bylayer, make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def file_bytes(path):
    with open(path, "rb") as f:
        return f.read()


@pytest.mark.parametrize("name,kw", [("tiny", dict(n_elems=1 << 18)), ("mlr", dict(rows=7)), ("mf", dict(l_rows=4000, r_rows=200)),
                                      ("lda", dict(vocab=1500))])
def test_stored_checkpoint_follows_the_oracle_and_serves_a_recovery(tmp_path, name, kw):
    w = make_workload(name, **kw)
    boff = block_offsets(w.geom)
    nb = boff.size - 1
    is_float = w.x.dtype == np.float32
    path = str(tmp_path / "running.ckpt")
    fd = os.open(path, os.O_RDWR | os.O_CREAT, 0o600)
    r = rng(70)
    hx = w.z.copy()  # training starts at x^(0), which is also the first running checkpoint (Section 4.2)
    xd = parity.to_dev(hx)
    ck = api.ScarCheckpoint(xd, n_shards=8, row_elems=w.geom.row_elems, block_elems=w.geom.block_elems)
    ck.store_full(fd)
    assert file_bytes(path) == hx.tobytes()
    k = max(1, nb // 6)
    max_len = int(np.diff(boff.astype(np.int64)).max())
    ck.drain_init(k, k * max_len)
    hz = hx.copy()
    for it in range(5):
        # one "iteration": parameters move, then a partial checkpoint goes to storage in the background
        if is_float:
            hx = (hx + r.standard_normal(hx.size).astype(np.float32) * np.repeat(r.lognormal(-2, 1, nb), np.diff(boff.astype(np.int64))).astype(np.float32)).astype(np.float32)
        else:
            hx = np.maximum(hx + r.integers(-2, 3, size=hx.size), 0).astype(np.int32)
        xd.copy_(torch.from_numpy(hx))
        ora = oracle.priority_save(hx, hz, boff, k=k)
        got = parity.check_save(ck, ck.priority_save_k(k), hx, hz, boff, ora)
        hz = parity.next_checkpoint(hz, hx, boff, got, ora)
        t = ck.drain_enqueue()
        ck.store_drained(t, fd)
        ck.drain_release(t)
        assert file_bytes(path) == hz.tobytes(), f"stored checkpoint differs after save {it}"
    os.fsync(fd)
    ck.close()
    # a failure: half of the shards lose their parameters; a new process recovers them from storage
    lost_shards = np.array([1, 0, 1, 0, 0, 1, 1, 0], dtype=np.uint8)
    lost = oracle.expand_shards(nb, lost_shards)
    x_now = hx.copy()
    want, x_after = oracle.recover_partial(x_now, hz, boff, lost)
    xd2 = parity.to_dev(x_now)
    ck2 = api.ScarCheckpoint(xd2, n_shards=8, row_elems=w.geom.row_elems, block_elems=w.geom.block_elems)
    ck2.load_stored(fd)
    assert parity.same_bits(ck2.views()["z"].cpu().numpy(), hz)
    parity.check_norm(ck2.recover_partial(lost_shards), want, is_float)
    assert xd2.cpu().numpy().tobytes() == x_after.tobytes()
    ck2.close()
    os.close(fd)


def test_stored_checkpoint_with_explicit_offsets_and_io_errors(tmp_path):
    boff, z, x = make_cnn_bylayer(scale=1, pad_to=1, dtype="f32", seed=8)
    nb = boff.size - 1
    path = str(tmp_path / "bylayer.ckpt")
    fd = os.open(path, os.O_RDWR | os.O_CREAT, 0o600)
    xd = parity.to_dev(x)
    ck = parity.make_ctx(xd, z, boff=boff, n_shards=1)
    ck.store_full(fd)
    assert file_bytes(path) == z.tobytes()
    lens = np.sort(np.diff(boff.astype(np.int64)))[::-1]
    ck.drain_init(nb, int(lens[0] + lens[1] - 1))
    with pytest.raises(api.ScarError) as e:
        ck.priority_save_k(2)  # the capacity rule: the k longest blocks of the layout must fit the slot
    assert e.value.code == -7
    ora = oracle.priority_save(x, z, boff, k=1)
    parity.check_save(ck, ck.priority_save_k(1), x, z, boff, ora)
    t = ck.drain_enqueue()
    ck.store_drained(t, fd)
    assert file_bytes(path) == ora.z_after.tobytes()
    # errors: a descriptor that cannot be written, a file that is too short to load
    ro = os.open(path, os.O_RDONLY)
    with pytest.raises(api.ScarError) as e:
        ck.store_drained(t, ro)
    assert e.value.code == -8
    os.close(ro)
    ck.drain_release(t)
    short = str(tmp_path / "short.ckpt")
    with open(short, "wb") as f:
        f.write(z.tobytes()[:1000])
    sfd = os.open(short, os.O_RDONLY)
    with pytest.raises(api.ScarError) as e:
        ck.load_stored(sfd)
    assert e.value.code == -8
    os.close(sfd)
    with pytest.raises(api.ScarError):
        ck.store_full(-1)
    ck.load_stored(fd)  # the context is still usable
    assert parity.same_bits(ck.views()["z"].cpu().numpy(), ora.z_after)
    ck.close()
    os.close(fd)
