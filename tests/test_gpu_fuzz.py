"""Randomised GPU parity: many small cases with random geometry (implicit and explicit, aligned or not, short,
long and empty blocks), element type, norm, selector, k and lost set, each compared with the oracle in full."""

import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def random_case(r):
    """Returns (kwargs for ScarCheckpoint, boff, x, z, norm name, weights or None)."""
    kind = r.choice(["implicit", "rows", "explicit", "explicit_long"])
    align = int(r.choice([1, 4]))
    if kind == "implicit":
        blk = int(r.integers(1, 600)) * align
        n = blk * int(r.integers(1, 300)) + (int(r.integers(0, blk)) // align * align if r.random() < 0.5 else 0)
        n = max(n, align)
        layout = dict(row_elems=0, block_elems=blk)
        boff = oracle.layout_offsets(n, 0, blk)
    elif kind == "rows":
        blk = int(r.integers(1, 200)) * align
        row = int(r.integers(1, 2000)) * align
        n = row * int(r.integers(1, 60))
        layout = dict(row_elems=row, block_elems=blk)
        boff = oracle.layout_offsets(n, row, blk)
    elif kind == "explicit":
        lens = r.integers(0, 500, size=int(r.integers(1, 400))) * align
        lens[r.random(lens.size) < 0.1] = 0
        if lens.sum() == 0:
            lens[0] = 4
        boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
        layout = dict(block_offsets=boff)
        n = int(boff[-1])
    else:  # a few very long blocks among short ones: the segmented path
        lens = r.integers(0, 300, size=int(r.integers(2, 40))) * align
        for i in r.choice(lens.size, size=min(3, lens.size), replace=False):
            lens[i] = int(r.integers(8193, 60000)) // align * align
        boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
        layout = dict(block_offsets=boff)
        n = int(boff[-1])
    nb = boff.size - 1
    lens = np.diff(boff.astype(np.int64))
    if r.random() < 0.35:
        z = r.poisson(3.0, size=n).astype(np.int32)
        x = np.maximum(z + r.integers(-3, 4, size=n) * (r.random(n) < 0.3), 0).astype(np.int32)
        norm, w = "l1i", None
    else:
        z = r.standard_normal(n).astype(np.float32)
        scale = np.repeat(r.lognormal(-1, 1.5, nb) * (r.random(nb) < 0.8), lens).astype(np.float32)
        x = (z + r.standard_normal(n).astype(np.float32) * scale).astype(np.float32)
        norm = str(r.choice(["l2", "l1"]))
        w = r.uniform(0, 3, nb).astype(np.float32) if r.random() < 0.4 else None
    layout["n_shards"] = int(r.integers(1, 12))
    return layout, boff, x, z, norm, w


def oracle_save(x, z, boff, k, norm, w):
    if norm in ("l1i",) or (norm == "l2" and w is None):
        return oracle.priority_save(x, z, boff, k=k)
    return oracle.save_norm(x, z, boff, k, norm, None if w is None else w.astype(np.float64))


def oracle_norm(x, z, boff, lost, norm, w):
    if norm in ("l1i",) or (norm == "l2" and w is None):
        return oracle.perturbation_norm(x, z, boff, lost)
    return oracle.perturbation_norm_weighted(x, z, boff, lost, norm, w)


@pytest.mark.parametrize("seed", range(256))
def test_random_case(seed):
    r = rng(1000 + seed)
    layout, boff, x, z, norm, w = random_case(r)
    nb = boff.size - 1
    is_float = x.dtype == np.float32
    xd = parity.to_dev(x)
    ck = api.ScarCheckpoint(xd, guarded=True, **layout)  # every library buffer between two guard bands
    assert ck.n_blocks == nb
    ck.load(parity.to_dev(z))
    if norm == "l1" or w is not None:
        ck.set_norm(api.SCAR_NORM_L1 if norm == "l1" else api.SCAR_NORM_DEFAULT, w)
    linear = norm == "l1"
    hz, cursor = z.copy(), 0
    for step in range(3):
        k = int(r.choice([0, 1, nb, int(r.integers(0, nb + 1))]))
        which = str(r.choice(["priority", "priority", "round", "random"]))
        if which == "priority":
            ora = oracle_save(x, hz, boff, k, norm, w)
            got = parity.check_save(ck, ck.priority_save_k(k), x, hz, boff, ora, linear=linear)
            hz = parity.next_checkpoint(hz, x, boff, got, ora)
        else:
            if which == "round":
                sel, cursor = oracle.select_round(nb, k, cursor)
                info = ck.save_round(k)
            else:
                pri = r.integers(0, int(r.choice([3, 2**32])), size=nb, dtype=np.uint64).astype(np.uint32)
                sel = oracle.select_random(pri, k)
                info = ck.save_random(k, parity.to_dev(pri.view(np.int32)))
            ora = oracle.save_selected(x, hz, boff, sel)
            got = parity.fetch_save(ck, info)
            assert int(info.k) == k and int(info.payload_elems) == ora.payload.size
            np.testing.assert_array_equal(got["sel"], ora.sel)
            np.testing.assert_array_equal(got["poff"], ora.poff)
            assert parity.same_bits(got["payload"], ora.payload) and parity.same_bits(got["z"], ora.z_after)
            hz = ora.z_after
        assert ck.round_cursor() == cursor
    # recovery from the checkpoint as it stands now
    parity.check_norm(ck.perturbation_norm(None), oracle_norm(x, hz, boff, None, norm, w), is_float)
    if r.random() < 0.5:
        shards = (r.random(layout["n_shards"]) < 0.4).astype(np.uint8)
        lost = oracle.expand_shards(nb, shards)
        parity.check_norm(ck.perturbation_norm(shards), oracle_norm(x, hz, boff, lost, norm, w), is_float)
        got_n = ck.recover_partial(shards)
    else:
        lost = (r.random(nb) < r.random()).astype(np.uint8)
        md = parity.to_dev(lost)
        parity.check_norm(ck.perturbation_norm_blocks(md), oracle_norm(x, hz, boff, lost, norm, w), is_float)
        got_n = ck.recover_partial_blocks(md)
    parity.check_norm(got_n, oracle_norm(x, hz, boff, lost, norm, w), is_float)
    _, x_after = oracle.recover_partial(x, hz, boff, lost)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    assert parity.same_bits(ck.views()["z"].cpu().numpy(), hz)
    assert ck.check_guards() == 0, "a kernel wrote just outside one of the library's buffers"
    ck.close()
