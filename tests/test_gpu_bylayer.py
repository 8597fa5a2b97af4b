"""GPU parity on layouts with very long and very unequal blocks (by-layer partitioning of a network,
Section 5.1), which the library cuts into segments: all four element paths (float / int, 16-byte aligned or
not), every strategy, recovery by shards and by block mask."""

import numpy as np
import pytest

import oracle
from workloads import make_cnn_bylayer

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


@pytest.mark.parametrize("dtype,pad_to", [("f32", 1), ("f32", 4), ("i32", 1), ("i32", 4)])
def test_bylayer_save_and_recovery(dtype, pad_to):
    boff, z, x = make_cnn_bylayer(scale=1, pad_to=pad_to, dtype=dtype, seed=5)
    nb = boff.size - 1
    assert nb == 10 and int(np.diff(boff.astype(np.int64)).max()) == 49 * 64 * 1024  # 3.2 M elements in one block
    is_float = dtype == "f32"
    for k in (0, 1, 3, nb):
        xd = parity.to_dev(x)
        ck = parity.make_ctx(xd, z, boff=boff, n_shards=5)
        ora = oracle.priority_save(x, z, boff, k=k)
        info = ck.priority_save_k(k)
        parity.check_save(ck, info, x, z, boff, ora)
        assert xd.cpu().numpy().tobytes() == x.tobytes()
        ck.close()
    xd = parity.to_dev(x)
    ck = parity.make_ctx(xd, z, boff=boff, n_shards=5)
    parity.check_norm(ck.perturbation_norm(None), oracle.perturbation_norm(x, z, boff, None), is_float)
    shards = np.array([0, 1, 0, 1, 0], dtype=np.uint8)  # layers 2,3 and 6,7: one conv and one fc layer
    lost = oracle.expand_shards(nb, shards)
    want, x_after = oracle.recover_partial(x, z, boff, lost)
    parity.check_norm(ck.perturbation_norm(shards), want, is_float)
    parity.check_norm(ck.recover_partial(shards), want, is_float)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    again = ck.recover_partial(shards)
    assert again.l2 == 0.0 and again.l1 == 0
    # arbitrary block mask on what is left
    lost2 = np.array([1, 1, 0, 0, 1, 0, 0, 0, 1, 1], dtype=np.uint8)
    want2, x_after2 = oracle.recover_partial(x_after, z, boff, lost2)
    parity.check_norm(ck.recover_partial_blocks(parity.to_dev(lost2)), want2, is_float)
    assert xd.cpu().numpy().tobytes() == x_after2.tobytes()
    assert parity.same_bits(ck.views()["z"].cpu().numpy(), z)
    ck.close()


def test_bylayer_strategies_and_sequence():
    boff, z0, x = make_cnn_bylayer(scale=1, pad_to=4, dtype="f32", seed=6)
    nb = boff.size - 1
    xd = parity.to_dev(x)
    ck = parity.make_ctx(xd, z0, boff=boff, n_shards=1)
    z, cur, r = z0.copy(), 0, rng(8)
    for step in range(6):
        if step % 3 == 0:
            sel, cur = oracle.select_round(nb, 4, cur)
            ora = oracle.save_selected(x, z, boff, sel)
            info = ck.save_round(4)
        elif step % 3 == 1:
            pri = r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32)
            ora = oracle.save_selected(x, z, boff, oracle.select_random(pri, 3))
            info = ck.save_random(3, parity.to_dev(pri.view(np.int32)))
        else:
            ora = oracle.priority_save(x, z, boff, k=2)
            info = ck.priority_save_k(2)
            parity.check_save(ck, info, x, z, boff, ora)
        got = parity.fetch_save(ck, info)
        np.testing.assert_array_equal(got["sel"], ora.sel)
        np.testing.assert_array_equal(got["poff"], ora.poff)
        assert parity.same_bits(got["payload"], ora.payload) and parity.same_bits(got["z"], ora.z_after)
        z = ora.z_after
        x = (x + r.standard_normal(x.size).astype(np.float32) * np.float32(1e-3)).astype(np.float32)
        xd.copy_(torch.from_numpy(x))
    ck.close()


def test_bylayer_weighted_l1_and_mixed_with_small_blocks():
    """Long blocks next to many short ones (embedding-like rows after a big matrix), weighted l1 norm."""
    r = rng(9)
    lens = np.concatenate([[200000, 37], r.integers(1, 400, size=500), [131072 + 5, 0, 90001]])
    boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    n, nb = int(boff[-1]), lens.size
    z = r.standard_normal(n).astype(np.float32)
    x = (z + r.standard_normal(n).astype(np.float32) * np.repeat(r.lognormal(-2, 1, nb), lens).astype(np.float32)).astype(np.float32)
    w = r.uniform(0.1, 2.0, nb).astype(np.float32)
    xd = parity.to_dev(x)
    ck = parity.make_ctx(xd, z, boff=boff, n_shards=4)
    ck.set_norm(api.SCAR_NORM_L1, w)
    ora = oracle.save_norm(x, z, boff, 100, "l1", w.astype(np.float64))
    parity.check_save(ck, ck.priority_save_k(100), x, z, boff, ora, linear=True)
    ck.load(parity.to_dev(z))
    lost = (r.random(nb) < 0.5).astype(np.uint8)
    lost[0] = 1
    want = oracle.perturbation_norm_weighted(x, z, boff, lost, "l1", w)
    parity.check_norm(ck.recover_partial_blocks(parity.to_dev(lost)), want, True)
    _, x_after = oracle.recover_partial(x, z, boff, lost)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    ck.close()


def test_implicit_layout_with_huge_blocks_uses_the_same_path():
    n, blk = 3 * 100000 * 4, 100000  # rows of 400 000 cut into blocks of 100 000: 12 blocks, each > 2 segments
    r = rng(10)
    z = r.standard_normal(n).astype(np.float32)
    x = (z + r.standard_normal(n).astype(np.float32) * np.float32(0.01)).astype(np.float32)
    x[5 * blk:6 * blk] = z[5 * blk:6 * blk]  # one untouched block: exact zero
    boff = oracle.layout_offsets(n, 400000, blk)
    xd = parity.to_dev(x)
    ck = api.ScarCheckpoint(xd, n_shards=3, row_elems=400000, block_elems=blk)
    ck.load(parity.to_dev(z))
    ora = oracle.priority_save(x, z, boff, k=5)
    got = parity.check_save(ck, ck.priority_save_k(5), x, z, boff, ora)
    assert got["scores"][5] == 0.0
    shards = np.array([1, 0, 1], dtype=np.uint8)
    want, x_after = oracle.recover_partial(x, parity.next_checkpoint(z, x, boff, got, ora), boff, oracle.expand_shards(12, shards))
    parity.check_norm(ck.recover_partial(shards), want, True)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    ck.close()
