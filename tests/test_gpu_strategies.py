"""GPU parity of the baseline selectors of Section 5.4 (`round`, `random`) against the CPU oracle.

Everything here is integer or byte work, so every comparison is bit-exact: ids, offsets, payload bytes,
refreshed checkpoint, cursor."""

import numpy as np
import pytest

import oracle
from workloads import Geometry, block_offsets, make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def check_exact(ck, info, ora, x_dev, x_host):
    assert int(info.k) == ora.k and int(info.nonfinite_blocks) == 0
    assert int(info.payload_elems) == ora.payload.size
    got = parity.fetch_save(ck, info)
    np.testing.assert_array_equal(got["sel"], ora.sel)
    np.testing.assert_array_equal(got["poff"], ora.poff)
    assert parity.same_bits(got["payload"], ora.payload), "payload bytes"
    assert parity.same_bits(got["z"], ora.z_after), "refreshed checkpoint"
    assert x_dev.cpu().numpy().tobytes() == x_host.tobytes(), "a save must not touch x"


def small_workload(name):
    sizes = {"tiny": dict(n_elems=1 << 18), "mlr": dict(rows=6), "mf": dict(l_rows=5000, r_rows=300),
             "lda": dict(vocab=3000)}
    return make_workload(name, **sizes[name])


@pytest.mark.parametrize("name", ["tiny", "mlr", "mf", "lda"])
def test_round_robin_sequence_with_wraps(name):
    w = small_workload(name)
    boff = block_offsets(w.geom)
    nb = boff.size - 1
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    z, cur = w.z.copy(), 0
    assert ck.round_cursor() == 0
    # k chosen so that the cursor wraps inside a save several times, with uneven steps
    for k in (nb // 3, nb // 3 + 5, nb // 2, 1, 0, nb // 7, nb - 1, nb):
        sel, nxt = oracle.select_round(nb, k, cur)
        ora = oracle.save_selected(w.x, z, boff, sel)
        info = ck.save_round(k)
        check_exact(ck, info, ora, xd, w.x)
        z, cur = ora.z_after, nxt
        assert ck.round_cursor() == cur
    ck.close()


def test_round_robin_cursor_set_and_full_cycle_is_a_full_checkpoint():
    w = make_workload("tiny", n_elems=1 << 16)
    boff = block_offsets(w.geom)
    nb = boff.size - 1
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    assert ck.round_cursor(nb - 3) == nb - 3
    sel, nxt = oracle.select_round(nb, 10, nb - 3)
    info = ck.save_round(10)
    check_exact(ck, info, oracle.save_selected(w.x, w.z, boff, sel), xd, w.x)
    assert ck.round_cursor() == nxt == 7
    with pytest.raises(api.ScarError):
        ck.round_cursor(nb)
    with pytest.raises(api.ScarError):
        ck.save_round(nb + 1)
    # one cycle of ceil(B/k) saves refreshes everything: perturbation 0 afterwards (Section 4: full checkpoint)
    ck.round_cursor(0)
    for _ in range(-(-nb // 100)):
        ck.save_round(100, sync=False)
    assert ck.perturbation_norm(None).l2 == 0.0
    assert ck.views()["z"].cpu().numpy().tobytes() == w.x.tobytes()
    ck.close()


@pytest.mark.parametrize("name", ["tiny", "mlr", "mf", "lda"])
def test_random_selector_distinct_and_tied_priorities(name):
    w = small_workload(name)
    boff = block_offsets(w.geom)
    nb = boff.size - 1
    r = rng(21)
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    z = w.z.copy()
    cases = [(r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32), nb // 4),
             (r.integers(0, 50, size=nb, dtype=np.uint64).astype(np.uint32), nb // 3),      # heavy ties
             (np.full(nb, 0xFFFFFFFF, dtype=np.uint32), nb // 5),                           # all equal: first ids
             (np.zeros(nb, dtype=np.uint32), 7),
             ((r.integers(0, 2**32, size=nb, dtype=np.uint64) | 0x7F800000).astype(np.uint32), nb // 2),  # no float meaning
             (r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32), 0),
             (r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32), nb)]
    for pri, k in cases:
        sel = oracle.select_random(pri, k)
        ora = oracle.save_selected(w.x, z, boff, sel)
        pd = parity.to_dev(pri.view(np.int32))
        info = ck.save_random(k, pd)
        check_exact(ck, info, ora, xd, w.x)
        z = ora.z_after
    ck.close()


def test_strategies_on_an_explicit_ragged_layout_and_interleaved_with_priority():
    r = rng(22)
    lens = r.integers(0, 70, size=3000)
    boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    n = int(boff[-1])
    z0 = r.standard_normal(n).astype(np.float32)
    x = (z0 + r.standard_normal(n).astype(np.float32) * 0.1).astype(np.float32)
    nb = boff.size - 1
    xd = parity.to_dev(x)
    ck = parity.make_ctx(xd, z0, boff=boff)
    z, cur = z0.copy(), 0
    for step in range(6):
        if step % 3 == 0:
            sel, cur = oracle.select_round(nb, 700, cur)
            ora = oracle.save_selected(x, z, boff, sel)
            info = ck.save_round(700)
            check_exact(ck, info, ora, xd, x)
        elif step % 3 == 1:
            pri = r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32)
            ora = oracle.save_selected(x, z, boff, oracle.select_random(pri, 500))
            info = ck.save_random(500, parity.to_dev(pri.view(np.int32)))
            check_exact(ck, info, ora, xd, x)
        else:
            ora = oracle.priority_save(x, z, boff, k=400)
            info = ck.priority_save_k(400)
            parity.check_save(ck, info, x, z, boff, ora)
        z = ora.z_after
    ck.close()


def test_full_size_cnn_round_and_random_properties():
    """At the benchmark's size the oracle's pack is replaced by what is unique at any size: the id list
    (computed by the oracle's selectors, which only see B, k, the cursor or the priorities) and sampled blocks."""
    n, blk = 1 << 30, 4096
    nb = n // blk
    g = torch.Generator(device="cuda").manual_seed(4)
    z0 = torch.randn(n, device="cuda", generator=g) * 5e-2
    x = z0 + torch.randn(n, device="cuda", generator=g) * 1e-4
    ck = api.ScarCheckpoint(x, n_shards=8, block_elems=blk)
    ck.load(z0)
    k = 26214
    ck.round_cursor(nb - 1000)
    sel, nxt = oracle.select_round(nb, k, nb - 1000)
    info = ck.save_round(k)
    v = ck.views(k, int(info.payload_elems))
    assert int(info.k) == k and int(info.payload_elems) == k * blk and ck.round_cursor() == nxt
    np.testing.assert_array_equal(v["sel"].cpu().numpy().view(np.uint32), sel)
    np.testing.assert_array_equal(v["poff"].cpu().numpy().view(np.uint64), np.arange(k + 1, dtype=np.uint64) * blk)
    pri = torch.randint(0, 2**31 - 1, (nb,), device="cuda", generator=g, dtype=torch.int32)
    sel2 = oracle.select_random(pri.cpu().numpy().view(np.uint32), k)
    info = ck.save_random(k, pri)
    v = ck.views(k, int(info.payload_elems))
    np.testing.assert_array_equal(v["sel"].cpu().numpy().view(np.uint32), sel2)
    # sampled blocks: payload and refreshed checkpoint hold x; untouched blocks still hold z0
    r = rng(5)
    taken = np.union1d(sel, sel2)
    for j in r.integers(0, k, size=64):
        b = int(sel2[j])
        assert torch.equal(v["payload"][j * blk:(j + 1) * blk], x[b * blk:(b + 1) * blk])
        assert torch.equal(v["z"][b * blk:(b + 1) * blk], x[b * blk:(b + 1) * blk])
    rest = np.setdiff1d(np.arange(nb), taken)
    for b in r.choice(rest, size=64, replace=False):
        b = int(b)
        assert torch.equal(v["z"][b * blk:(b + 1) * blk], z0[b * blk:(b + 1) * blk])
    ck.close()
