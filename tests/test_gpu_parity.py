"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs, through the C ABI."""

import ctypes as C

import numpy as np
import pytest

import oracle
from workloads import Geometry, block_offsets, make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402  (tests/parity.py)
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def run_save_and_recover(w, r_values, boff=None, n_shards=None, lost_blocks=None, lost_shards=None):
    """Full protocol on one workload: every r (each from the pristine state), what-if norm, recovery."""
    explicit = boff is not None
    boff = boff if explicit else block_offsets(w.geom)
    is_float = w.x.dtype == np.float32
    for r in r_values:
        xd = parity.to_dev(w.x)
        ck = parity.make_ctx(xd, w.z, geom=w.geom, boff=boff if explicit else None, n_shards=n_shards or 8)
        assert ck.n_blocks == boff.size - 1
        ora = oracle.priority_save(w.x, w.z, boff, r=r)
        info = ck.priority_save(r)
        parity.check_save(ck, info, w.x, w.z, boff, ora)
        assert torch.equal(xd.cpu(), torch.from_numpy(w.x)), "a save must not touch x"
        ck.close()
    # recovery legs from the pristine state
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom, boff=boff if explicit else None, n_shards=n_shards or 8)
    full = ck.perturbation_norm(None)
    parity.check_norm(full, oracle.perturbation_norm(w.x, w.z, boff, None), is_float)
    lost_blocks = lost_blocks if lost_blocks is not None else w.lost_blocks
    lost_shards = lost_shards if lost_shards is not None else w.lost_shards
    if lost_shards is not None:
        lb = oracle.expand_shards(boff.size - 1, lost_shards)
        ora_n, x_after = oracle.recover_partial(w.x, w.z, boff, lb)
        parity.check_norm(ck.perturbation_norm(lost_shards), ora_n, is_float)
        assert torch.equal(xd.cpu(), torch.from_numpy(w.x)), "the what-if norm must not write"
        got = ck.recover_partial(lost_shards)
    else:
        lb = lost_blocks
        ora_n, x_after = oracle.recover_partial(w.x, w.z, boff, lb)
        md = parity.to_dev(lb)
        parity.check_norm(ck.perturbation_norm_blocks(md), ora_n, is_float)
        got = ck.recover_partial_blocks(md)
    parity.check_norm(got, ora_n, is_float)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes(), "restored buffer differs from the oracle's"
    assert ck.views()["z"].cpu().numpy().tobytes() == w.z.tobytes(), "recovery must not touch z"
    # idempotence: nothing left to restore
    again = ck.recover_partial(lost_shards) if lost_shards is not None else ck.recover_partial_blocks(md)
    assert again.l2 == 0.0 and again.l1 == 0
    ck.close()


# ------------------------------------------------------------------ the five configurations


def test_tiny_full_size():
    w = make_workload("tiny")
    assert w.n_blocks == 4096
    run_save_and_recover(w, w.r_values)


def test_mlr_full_size():
    w = make_workload("mlr")
    assert w.n_blocks == 98_000
    run_save_and_recover(w, w.r_values)


def test_mf_full_size():
    w = make_workload("mf")
    assert w.n_blocks == 498_000
    run_save_and_recover(w, w.r_values)


def test_lda_full_size_bit_exact():
    w = make_workload("lda")
    assert w.n_blocks == 100_000 and w.x.dtype == np.int32
    run_save_and_recover(w, w.r_values)


def test_cnn_reduced_all_r():
    w = make_workload("cnn", n_elems=1 << 25)
    assert w.n_blocks == 8192
    run_save_and_recover(w, w.r_values)


def test_cnn_full_size_in_the_benchmark_configuration():
    """2**30 elements, 262 144 blocks of 4096, 8 shards: the launch configuration bench.py times.

    The parameter set comes from the seeded device generator the benchmark uses; the oracle gets the
    same bytes through a device-to-host copy and is run in full (about 10 s of CPU time per sweep)."""
    from workloads.configs import make_cnn_device

    geom, z_dev, x_dev, lost_shards = make_cnn_device(1 << 30, 4096, seed=4, device="cuda:0")
    x_host, z_host = x_dev.cpu().numpy(), z_dev.cpu().numpy()
    boff = block_offsets(geom)
    ck = api.ScarCheckpoint(x_dev, n_shards=8, block_elems=4096)
    assert ck.n_blocks == 262_144
    for r, k in zip((0.01, 0.1, 0.5, 1.0), (2621, 26_214, 131_072, 262_144)):
        ck.load(z_dev)
        ora = oracle.priority_save(x_host, z_host, boff, r=r)
        assert ora.k == k
        info = ck.priority_save(r)
        parity.check_save(ck, info, x_host, z_host, boff, ora)
        del ora
    ck.load(z_dev)
    parity.check_norm(ck.perturbation_norm(None), oracle.perturbation_norm(x_host, z_host, boff, None), True)
    lb = oracle.expand_shards(262_144, lost_shards)
    ora_n, x_after = oracle.recover_partial(x_host, z_host, boff, lb)
    parity.check_norm(ck.recover_partial(lost_shards), ora_n, True)
    assert parity.same_bits(x_dev.cpu().numpy(), x_after), "restored buffer differs from the oracle's"
    assert ora_n.lost_elems == 1 << 27
    ck.close()


# ------------------------------------------------------------------ geometry variants and ragged tails


@pytest.mark.parametrize("n,row,blk", [
    (1 << 16, 0, 16), (1 << 16, 0, 64), (25_600, 100, 100), (1 << 18, 0, 1024), (1 << 20, 0, 65_536),
    (40_000, 10_000, 1024),  # tail of 784 per row
    (30_030, 10, 3),  # unaligned blocks of 3,3,3,1: element-wise path
    (70_000, 7_000, 999),  # unaligned, tail of 7
    (1 << 22, 0, 1 << 22),  # one giant block: exercises the fp64 flush
    (5, 0, 8),  # a single short block
])
@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_implicit_layouts(n, row, blk, kind):
    r = rng(n + blk)
    geom = Geometry(n, row, blk, 8)
    if kind == "f32":
        z = r.standard_normal(n).astype(np.float32)
        x = (z + r.standard_normal(n).astype(np.float32) * np.float32(0.01)).astype(np.float32)
    else:
        z = r.integers(-1000, 1000, size=n).astype(np.int32)
        x = (z + r.integers(-5, 6, size=n)).astype(np.int32)
    w = make_workload("tiny", n_elems=16)  # container only
    w.geom, w.x, w.z = geom, x, z
    w.lost_shards = np.array([0, 1, 0, 0, 1, 1, 0, 0], dtype=np.uint8)
    run_save_and_recover(w, (0.3,))


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_explicit_ragged_offsets_with_empty_blocks(seed, kind):
    r = rng(50 + seed)
    nb = 3000
    lens = r.integers(0, 300, size=nb)
    if seed == 2:
        lens = lens // 4 * 4  # all aligned: vector path with explicit offsets
    lens[r.integers(0, nb, size=50)] = 0
    boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    n = int(boff[-1])
    if kind == "f32":
        z = r.standard_normal(n).astype(np.float32)
        x = (z + r.standard_normal(n).astype(np.float32) * np.repeat(r.lognormal(0, 1, nb), lens).astype(np.float32)).astype(np.float32)
    else:
        z = r.poisson(3.0, size=n).astype(np.int32)
        x = np.maximum(z + r.integers(-2, 3, size=n), 0).astype(np.int32)
    w = make_workload("tiny", n_elems=16)
    w.x, w.z = x, z
    lost = (r.random(nb) < 0.3).astype(np.uint8)
    w.lost_shards = None
    run_save_and_recover(w, (0.1, 0.9), boff=boff, n_shards=5, lost_blocks=lost)
    w.lost_shards = np.array([1, 0, 0, 1, 0], dtype=np.uint8)
    run_save_and_recover(w, (), boff=boff, n_shards=5)


# ------------------------------------------------------------------ degenerate selections


@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_k_extremes_and_exact_ties(kind):
    w = make_workload("tiny", n_elems=1 << 16) if kind == "f32" else make_workload("lda", vocab=700, topics=120)
    boff = block_offsets(w.geom)
    nb = w.n_blocks
    for k in (0, 1, nb - 1, nb):
        xd = parity.to_dev(w.x)
        ck = parity.make_ctx(xd, w.z, geom=w.geom)
        ora = oracle.priority_save(w.x, w.z, boff, k=k)
        got = parity.check_save(ck, ck.priority_save_k(k), w.x, w.z, boff, ora)
        assert got["exact"]
        if k == nb:  # the traditional full checkpoint
            assert got["payload"].tobytes() == w.x.tobytes() and got["z"].tobytes() == w.x.tobytes()
        ck.close()
    # right after init every score is zero: ties go to the lowest ids
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, None, geom=w.geom)
    info = ck.priority_save_k(37)
    got = parity.fetch_save(ck, info)
    assert got["sel"].tolist() == list(range(37)) and not got["scores"].any()
    assert ck.perturbation_norm(None).l2 == 0.0
    ck.close()


def test_second_save_selects_what_is_left():
    w = make_workload("tiny", n_elems=1 << 16)
    boff = block_offsets(w.geom)
    k = w.n_blocks // 2 + 9
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    first = oracle.priority_save(w.x, w.z, boff, k=k)
    parity.check_save(ck, ck.priority_save_k(k), w.x, w.z, boff, first)
    second = oracle.priority_save(w.x, first.z_after, boff, k=k)
    got = parity.check_save(ck, ck.priority_save_k(k), w.x, first.z_after, boff, second)
    assert got["exact"] and got["z"].tobytes() == w.x.tobytes()
    ck.close()


def test_few_distinct_scores_many_ties():
    r = rng(7)
    nb, blk = 5000, 8
    geom = Geometry(nb * blk, 0, blk, 8)
    z = np.zeros(nb * blk, dtype=np.float32)
    x = z.copy()
    x[::blk] = r.integers(0, 4, size=nb).astype(np.float32)  # scores in {0, 1, 4, 9}
    boff = block_offsets(geom)
    for k in (1, 1234, 2500, 4999):
        xd = parity.to_dev(x)
        ck = parity.make_ctx(xd, z, geom=geom)
        ora = oracle.priority_save(x, z, boff, k=k)
        assert parity.check_save(ck, ck.priority_save_k(k), x, z, boff, ora)["exact"]
        ck.close()


@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_more_blocks_than_one_selection_tile_per_cta(kind):
    """Beyond 4096 blocks per SM the selection's CTAs walk several tiles each and re-read their keys (another
    kernel than the one-tile-per-CTA form): 700 000 blocks of 4 elements, many exact ties at zero, and a k that
    ends inside the ties."""
    r = rng(21)
    nb, blk = 700_000, 4
    geom = Geometry(nb * blk, 0, blk, 8)
    if kind == "f32":
        z = r.standard_normal(nb * blk).astype(np.float32)
        d = r.standard_normal(nb * blk).astype(np.float32) * np.repeat(r.lognormal(0, 1, nb), blk).astype(np.float32)
    else:
        z = r.integers(0, 50, size=nb * blk).astype(np.int32)
        d = r.integers(-3, 4, size=nb * blk).astype(np.int32)
    d.reshape(nb, blk)[r.random(nb) < 0.5] = 0  # half of the blocks unchanged: score exactly 0
    x = (z + d).astype(z.dtype)
    boff = block_offsets(geom)
    for k in (1, 70_001, 350_000 + 12_345, nb - 3):
        xd = parity.to_dev(x)
        ck = parity.make_ctx(xd, z, geom=geom)
        ora = oracle.priority_save(x, z, boff, k=k)
        parity.check_save(ck, ck.priority_save_k(k), x, z, boff, ora)
        ck.close()


@pytest.mark.parametrize("nb", [20_000, 650_000])
@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_ties_run_out_inside_one_cta_with_blocks_of_many_lengths(nb, kind):
    """Explicit ragged layout (block lengths 0..9, so every offset needs the lengths of what was taken before it),
    60 % of the blocks unchanged (score exactly 0), and k beyond the changed blocks: the k-th score is 0, the ties
    go to the lowest ids and run out inside one selection CTA; the CTAs behind it need the summed length of what
    it takes.  20 000 blocks: five CTAs of the one-tile kernel; 650 000: the several-tiles-per-CTA kernel."""
    r = rng(31 + nb)
    lens = r.integers(0, 10, size=nb)
    boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    n = int(boff[-1])
    changed = r.random(nb) < 0.4
    mask = np.repeat(changed, lens)
    if kind == "f32":
        z = r.standard_normal(n).astype(np.float32)
        x = (z + mask * r.standard_normal(n).astype(np.float32)).astype(np.float32)
    else:
        z = r.integers(0, 100, size=n).astype(np.int32)
        x = (z + mask * r.integers(1, 5, size=n)).astype(np.int32)
    n_changed = int(((lens > 0) & changed).sum())
    for k in (n_changed + nb // 5, n_changed + 1, nb - 1):
        xd = parity.to_dev(x)
        ck = parity.make_ctx(xd, z, boff=boff, n_shards=4)
        ora = oracle.priority_save(x, z, boff, k=k)
        got = parity.check_save(ck, ck.priority_save_k(k), x, z, boff, ora)
        assert got["exact"], "ties at exactly zero leave no freedom"
        ck.close()


@pytest.mark.parametrize("rows", [600, 4_000, 140_000])
@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_ties_run_out_on_rows_with_a_short_last_block(rows, kind):
    """Implicit layout whose rows end in a shorter block (five blocks per row: 8, 8, 8, 8, 5 elements), which the
    selection treats as a layout of two block lengths; 60 % of the blocks unchanged, k beyond the changed ones, so
    the ties at zero run out inside one selection CTA and every offset behind depends on which lengths were taken.
    600 rows: one CTA; 4000 rows: five CTAs of the one-tile kernel; 140 000 rows: several tiles per CTA."""
    r = rng(77 + rows)
    row, blk = 37, 8
    n, nb = rows * row, rows * 5
    geom = Geometry(n, row, blk, 4)
    boff = block_offsets(geom)
    lens = np.diff(boff.astype(np.int64))
    changed = r.random(nb) < 0.4
    mask = np.repeat(changed, lens)
    if kind == "f32":
        z = r.standard_normal(n).astype(np.float32)
        x = (z + mask * r.standard_normal(n).astype(np.float32)).astype(np.float32)
    else:
        z = r.integers(0, 100, size=n).astype(np.int32)
        x = (z + mask * r.integers(1, 5, size=n)).astype(np.int32)
    n_changed = int(changed.sum())
    for k in (n_changed + nb // 5, n_changed + 1, nb - 1):
        xd = parity.to_dev(x)
        ck = parity.make_ctx(xd, z, geom=geom)
        ora = oracle.priority_save(x, z, boff, k=k)
        got = parity.check_save(ck, ck.priority_save_k(k), x, z, boff, ora)
        assert got["exact"], "ties at exactly zero leave no freedom"
        ck.close()


def test_uint64_keys_above_32_bits():
    r = rng(8)
    nb, blk = 4000, 16
    geom = Geometry(nb * blk, 0, blk, 8)
    z = np.full(nb * blk, np.iinfo(np.int32).min, dtype=np.int32)
    x = z.copy()
    big = r.random(nb) < 0.4
    xv = x.reshape(nb, blk)
    xv[big, : 8] = np.iinfo(np.int32).max  # block score 8 * (2^32 - 1) > 2^32
    xv[~big, 0] += r.integers(0, 1000, size=(~big).sum()).astype(np.int32)
    boff = block_offsets(geom)
    for k in (5, int(big.sum()), int(big.sum()) + 17):
        xd = parity.to_dev(x)
        ck = parity.make_ctx(xd, z, geom=geom)
        ora = oracle.priority_save(x, z, boff, k=k)
        assert ora.scores.max() > 2 ** 32
        parity.check_save(ck, ck.priority_save_k(k), x, z, boff, ora)
        # a later selection over small keys must not be confused by the large ones seen before
        ck.load(parity.to_dev(x))
        x2 = x.copy()
        x2[:: 3 * blk] += 1
        xd.copy_(torch.from_numpy(x2))
        ora2 = oracle.priority_save(x2, x, boff, k=11)
        parity.check_save(ck, ck.priority_save_k(11), x2, x, boff, ora2)
        ck.close()


def test_nonfinite_blocks_rank_first_and_survive_bitwise():
    w = make_workload("tiny", n_elems=1 << 14)
    x = w.x.copy()
    blk = w.geom.block_elems
    x.view(np.uint32)[5 * blk + 3] = 0x7FC00123  # NaN with a payload
    x[9 * blk] = np.inf
    x[20 * blk + 1] = -np.inf
    boff = block_offsets(w.geom)
    xd = parity.to_dev(x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    ora = oracle.priority_save(x, w.z, boff, k=5)
    assert ora.nonfinite_blocks == 3 and {5, 9, 20} <= set(ora.sel.tolist())
    got = parity.check_save(ck, ck.priority_save_k(5), x, w.z, boff, ora)
    assert got["exact"]
    n = ck.perturbation_norm(None)
    assert not np.isfinite(n.l2)
    ck.close()


# ------------------------------------------------------------------ recovery details


def test_masks_empty_full_and_more_shards_than_blocks():
    w = make_workload("tiny", n_elems=1 << 12, block_elems=512)  # 8 blocks
    boff = block_offsets(w.geom)
    xd = parity.to_dev(w.x)
    ck = api.ScarCheckpoint(xd, n_shards=13, block_elems=512)
    ck.load(parity.to_dev(w.z))
    none = np.zeros(13, dtype=np.uint8)
    res = ck.recover_partial(none)
    assert (res.l2, res.lost_blocks, res.lost_elems) == (0.0, 0, 0)
    assert xd.cpu().numpy().tobytes() == w.x.tobytes()
    for s in range(13):
        m = none.copy()
        m[s] = 200
        lb = oracle.expand_shards(8, m)
        parity.check_norm(ck.perturbation_norm(m), oracle.perturbation_norm(w.x, w.z, boff, lb), True)
    every = np.ones(13, dtype=np.uint8)
    ora_n, x_after = oracle.recover_partial(w.x, w.z, boff, np.ones(8, np.uint8))
    parity.check_norm(ck.recover_partial(every), ora_n, True)
    assert xd.cpu().numpy().tobytes() == w.z.tobytes() == x_after.tobytes()
    ck.close()


@pytest.mark.parametrize("n_shards,pattern", [(100, "alternate"), (64, "pairs"), (33, "alternate"), (7, "ends"),
                                              (3000, "alternate")])  # more shards than travel by value: staged copy
def test_many_lost_shard_runs(n_shards, pattern):
    # few runs travel inside the launch parameters, many fall back to a device-side block mask
    w = make_workload("tiny", n_elems=1 << 18, block_elems=64)  # 4096 blocks
    boff = block_offsets(w.geom)
    m = np.zeros(n_shards, dtype=np.uint8)
    if pattern == "alternate":
        m[::2] = 1
    elif pattern == "pairs":
        m[0::4] = 1
        m[1::4] = 1
    else:
        m[0] = m[-1] = 1
    xd = parity.to_dev(w.x)
    ck = api.ScarCheckpoint(xd, n_shards=n_shards, block_elems=64)
    ck.load(parity.to_dev(w.z))
    lb = oracle.expand_shards(w.n_blocks, m)
    ora_n, x_after = oracle.recover_partial(w.x, w.z, boff, lb)
    parity.check_norm(ck.perturbation_norm(m), ora_n, True)
    parity.check_norm(ck.recover_partial(m), ora_n, True)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    ck.close()


def test_recovery_does_not_write_outside_x():
    w = make_workload("mf", l_rows=4000, r_rows=150)
    n = w.x.size
    pad = 64
    buf = torch.full((n + 2 * pad,), 12345.0, dtype=torch.float32, device="cuda")
    xd = buf[pad: pad + n]
    xd.copy_(torch.from_numpy(w.x))
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    ck.recover_partial_blocks(parity.to_dev(w.lost_blocks))
    ck.priority_save(1.0)
    torch.cuda.synchronize()
    assert torch.all(buf[:pad] == 12345.0) and torch.all(buf[pad + n:] == 12345.0)
    ck.close()


def test_theorem_4_2_partition_identity_on_gpu():
    w = make_workload("tiny")
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    full = ck.perturbation_norm(None).l2 ** 2
    parts = 0.0
    for s in range(8):
        m = np.zeros(8, dtype=np.uint8)
        m[s] = 1
        part = ck.perturbation_norm(m)
        assert part.l2 <= ck.perturbation_norm(None).l2  # Theorem 4.1
        parts += part.l2 ** 2
    assert abs(parts - full) <= 1e-9 * full
    ck.close()


def test_results_are_bit_reproducible():
    w = make_workload("cnn", n_elems=1 << 24)
    outs = []
    for _ in range(3):
        xd = parity.to_dev(w.x)
        ck = parity.make_ctx(xd, w.z, geom=w.geom)
        info = ck.priority_save(0.1)
        got = parity.fetch_save(ck, info)
        nrm = ck.recover_partial(w.lost_shards)
        outs.append((got["scores"].tobytes(), got["sel"].tobytes(), got["payload"].tobytes(), nrm.l2))
        ck.close()
    assert outs[0] == outs[1] == outs[2]


# ------------------------------------------------------------------ host-buffer entry points, bookkeeping, errors


def test_host_buffer_entry_points():
    w = make_workload("mlr", rows=40, cols=10_000)
    boff = block_offsets(w.geom)
    n, nb = w.x.size, w.n_blocks
    xd = torch.zeros(n, dtype=torch.float32, device="cuda")
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    hx = torch.from_numpy(w.x).pin_memory()
    h_payload = torch.empty(n, dtype=torch.float32).pin_memory()
    h_sel = torch.empty(nb, dtype=torch.int32).pin_memory()
    h_poff = torch.empty(nb + 1, dtype=torch.int64).pin_memory()
    info = api.scar_ckpt_priority_save_host(ck.ctx, hx, 0.25, h_payload, h_sel, h_poff)
    ora = oracle.priority_save(w.x, w.z, boff, r=0.25)
    k = ora.k
    assert int(info.k) == k and int(info.payload_elems) == ora.payload.size
    if np.array_equal(h_sel.numpy()[:k].view(np.uint32), ora.sel):
        assert h_payload.numpy()[: ora.payload.size].tobytes() == ora.payload.tobytes()
        assert h_poff.numpy()[: k + 1].view(np.uint64).tolist() == ora.poff.tolist()
    parity.check_save(ck, info, w.x, w.z, boff, ora)
    # recovery through host buffers: only the lost ranges travel
    ck.load(parity.to_dev(w.z))
    hx2 = torch.from_numpy(w.x.copy()).pin_memory()
    lb = oracle.expand_shards(nb, w.lost_shards)
    ora_n, x_after = oracle.recover_partial(w.x, w.z, boff, lb)
    xd.zero_()  # device x is stale everywhere; the call must upload what it needs
    got = api.scar_recover_partial_host(ck.ctx, hx2, w.lost_shards)
    parity.check_norm(got, ora_n, True)
    assert hx2.numpy().tobytes() == x_after.tobytes()
    ck.close()


def test_launch_count_profile_and_last_info():
    w = make_workload("tiny", n_elems=1 << 16)
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    n0 = api.scar_ckpt_launch_count(ck.ctx)
    api.scar_ckpt_profile(ck.ctx, True)
    assert ck.priority_save(0.25, sync=False) is None
    n1 = api.scar_ckpt_launch_count(ck.ctx)
    assert n1 - n0 == 1 + 1 + 1  # scores, the one selection kernel, pack
    ms = api.scar_ckpt_profile_read(ck.ctx)
    assert ms[0] > 0 and ms[1] > 0 and ms[2] > 0 and ms[3] == 0 and ms[4] == 0
    ck.recover_partial(w.lost_shards, sync=False)
    assert api.scar_ckpt_launch_count(ck.ctx) - n1 == 1  # restore and norm reduction are one kernel
    ms = api.scar_ckpt_profile_read(ck.ctx)
    assert ms[3] > 0 and ms[4] >= 0 and ms[0] == 0
    s, nrm = api.scar_ckpt_last_info(ck.ctx)
    assert int(s.k) == 64 and int(nrm.lost_blocks) == 128
    ck.block_scores()
    torch.cuda.synchronize()
    api.scar_ckpt_profile(ck.ctx, False)
    ck.close()


def test_runtime_argument_errors():
    w = make_workload("tiny", n_elems=1 << 12)
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    lib = api.load_library()
    for bad in (-0.01, 1.01, float("nan")):
        assert lib.scar_ckpt_priority_save(ck.ctx, bad, None) == -1
    assert lib.scar_ckpt_priority_save_k(ck.ctx, ck.n_blocks + 1, None) == -1
    assert lib.scar_recover_partial(ck.ctx, None, None) == -1
    assert lib.scar_recover_partial_blocks(ck.ctx, None, None) == -1
    fresh = api.ScarCheckpoint(parity.to_dev(w.x), block_elems=256)
    assert lib.scar_ckpt_last_info(fresh.ctx, C.byref(api.scar_save_info()), None) == -5
    fresh.close()
    # nothing above changed any state
    ora = oracle.priority_save(w.x, w.z, block_offsets(w.geom), r=0.5)
    parity.check_save(ck, ck.priority_save(0.5), w.x, w.z, block_offsets(w.geom), ora)
    ck.close()


def test_empty_buffer():
    xd = torch.empty(0, dtype=torch.float32, device="cuda")
    ck = api.ScarCheckpoint(xd, n_shards=4, block_elems=256)
    assert ck.n_blocks == 0
    info = ck.priority_save(0.5)
    assert (int(info.k), int(info.payload_elems)) == (0, 0)
    n = ck.recover_partial(np.ones(4, np.uint8))
    assert (n.l2, int(n.lost_blocks)) == (0.0, 0)
    ck.close()


# ------------------------------------------------------------------ the bounded wait


@pytest.mark.parametrize("kind", ["f32", "i32"])
def test_a_barrier_that_cannot_complete_times_out_and_the_context_survives(kind):
    """The selection's grid barrier gives up after a bounded number of tries: the save reports a timeout, has
    copied nothing, and the next save is exact again.  The wait is made to run out by mis-setting what it
    waits for (one key more than exists: a condition that nothing fulfils), never by a fault."""
    w = make_workload("tiny", n_elems=1 << 20) if kind == "f32" else make_workload("lda", vocab=20_000, topics=100)
    boff = block_offsets(w.geom)
    xd = parity.to_dev(w.x)
    ck = parity.make_ctx(xd, w.z, geom=w.geom)
    k = w.n_blocks // 4
    api.scar_ckpt_selftest_arm_timeout(ck.ctx)
    with pytest.raises(api.ScarError) as e:
        ck.priority_save_k(k)
    assert e.value.code == -6 and "wait" in str(e.value)
    assert parity.same_bits(ck.views()["z"].cpu().numpy(), w.z), "a save that timed out must not touch z"
    assert xd.cpu().numpy().tobytes() == w.x.tobytes()
    ora = oracle.priority_save(w.x, w.z, boff, k=k)
    parity.check_save(ck, ck.priority_save_k(k), w.x, w.z, boff, ora)
    # armed again, read through last_info after an enqueue-only save; then a random save goes through
    api.scar_ckpt_selftest_arm_timeout(ck.ctx)
    ck.priority_save_k(k, sync=False)
    with pytest.raises(api.ScarError) as e:
        api.scar_ckpt_last_info(ck.ctx, True, False)
    assert e.value.code == -6
    pri = rng(3).integers(0, 2**32, size=w.n_blocks, dtype=np.uint64).astype(np.uint32)
    info = ck.save_random(5, parity.to_dev(pri.view(np.int32)))
    assert int(info.k) == 5
    np.testing.assert_array_equal(parity.fetch_save(ck, info)["sel"], oracle.select_random(pri, 5))
    ck.close()


def test_many_shard_runs_can_be_captured_and_replayed_with_the_mask_of_the_capture():
    """64 alternating lost shards do not fit the launch parameters as runs, so the shard flags travel by value
    inside the expansion kernel's parameters: nothing reads the caller's array after the call returns, and a
    captured recovery replays with the mask it was captured with even after that array has changed."""
    w = make_workload("tiny", n_elems=1 << 18, block_elems=64)  # 4096 blocks
    boff = block_offsets(w.geom)
    s = torch.cuda.Stream()
    x = parity.to_dev(w.x)
    x0 = x.clone()
    torch.cuda.synchronize()
    ck = api.ScarCheckpoint(x, n_shards=64, block_elems=64, stream=s)
    ck.load(parity.to_dev(w.z))
    torch.cuda.synchronize()
    m = np.zeros(64, dtype=np.uint8)
    m[::2] = 1
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        ck.recover_partial(m, sync=False)
    want, x_after = oracle.recover_partial(w.x, w.z, boff, oracle.expand_shards(w.n_blocks, m))
    m[:] = 0  # the caller's array is its own again
    for _ in range(2):
        x.copy_(x0)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        _, nrm = api.scar_ckpt_last_info(ck.ctx, False, True)
        parity.check_norm(nrm, want, True)
        assert x.cpu().numpy().tobytes() == x_after.tobytes()
    ck.close()


# ------------------------------------------------------------------ several contexts at once


def test_two_contexts_on_two_streams_run_side_by_side():
    """Each context has its own stream and its own work arrays; saves and recoveries enqueued on both without
    waiting in between (the selection kernels are cooperative launches that may have to take turns) give the same
    bytes as when each runs alone."""
    wa = make_workload("tiny", n_elems=1 << 22, seed=11)
    wb = make_workload("lda", vocab=30_000, topics=200, seed=12)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    xa, xb = parity.to_dev(wa.x), parity.to_dev(wb.x)
    za, zb = parity.to_dev(wa.z), parity.to_dev(wb.z)
    torch.cuda.synchronize()
    ca = api.ScarCheckpoint(xa, n_shards=8, block_elems=wa.geom.block_elems, stream=sa)
    cb = api.ScarCheckpoint(xb, n_shards=8, row_elems=wb.geom.row_elems, block_elems=wb.geom.block_elems, stream=sb)
    boa, bob = block_offsets(wa.geom), block_offsets(wb.geom)
    ka, kb = wa.n_blocks // 4, wb.n_blocks // 5
    ora_a = oracle.priority_save(wa.x, wa.z, boa, k=ka)
    ora_b = oracle.priority_save(wb.x, wb.z, bob, k=kb)
    for rep in range(5):
        ca.load(za)
        cb.load(zb)
        for _ in range(3):  # back-to-back saves on both streams, nothing waits
            ca.priority_save_k(ka, sync=False)
            cb.priority_save_k(kb, sync=False)
        ca.load(za)
        cb.load(zb)
        ca.priority_save_k(ka, sync=False)
        cb.priority_save_k(kb, sync=False)
        ia, _ = api.scar_ckpt_last_info(ca.ctx, True, False)
        ib, _ = api.scar_ckpt_last_info(cb.ctx, True, False)
        parity.check_save(ca, ia, wa.x, wa.z, boa, ora_a)
        parity.check_save(cb, ib, wb.x, wb.z, bob, ora_b)
    ca.load(za)
    cb.load(zb)
    ca.recover_partial(wa.lost_shards, sync=False)
    cb.recover_partial(wb.lost_shards, sync=False)
    _, na = api.scar_ckpt_last_info(ca.ctx, False, True)
    _, nb_ = api.scar_ckpt_last_info(cb.ctx, False, True)
    want_a, xa_after = oracle.recover_partial(wa.x, wa.z, boa, oracle.expand_shards(wa.n_blocks, wa.lost_shards))
    want_b, xb_after = oracle.recover_partial(wb.x, wb.z, bob, oracle.expand_shards(wb.n_blocks, wb.lost_shards))
    parity.check_norm(na, want_a, True)
    parity.check_norm(nb_, want_b, False)
    torch.cuda.synchronize()
    assert xa.cpu().numpy().tobytes() == xa_after.tobytes() and xb.cpu().numpy().tobytes() == xb_after.tobytes()
    ca.close()
    cb.close()


def test_enqueue_only_calls_can_be_captured_in_a_cuda_graph():
    """Calls with a NULL result pointer only enqueue, so a reload + save + recovery sequence can be captured once
    and replayed; every replay gives the oracle's bytes."""
    w = make_workload("tiny", n_elems=1 << 20)
    boff = block_offsets(w.geom)
    s = torch.cuda.Stream()
    x, z0 = parity.to_dev(w.x), parity.to_dev(w.z)
    x0 = x.clone()
    torch.cuda.synchronize()
    ck = api.ScarCheckpoint(x, n_shards=8, block_elems=w.geom.block_elems, stream=s)
    k = w.n_blocks // 4
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        ck.load(z0)
        ck.priority_save_k(k, sync=False)
        ck.recover_partial(w.lost_shards, sync=False)
    ora = oracle.priority_save(w.x, w.z, boff, k=k)
    lost = oracle.expand_shards(w.n_blocks, w.lost_shards)
    for _ in range(3):
        x.copy_(x0)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        info, nrm = api.scar_ckpt_last_info(ck.ctx)
        got = parity.check_save(ck, info, w.x, w.z, boff, ora)
        want, x_after = oracle.recover_partial(w.x, parity.next_checkpoint(w.z, w.x, boff, got, ora), boff, lost)
        parity.check_norm(nrm, want, True)
        assert x.cpu().numpy().tobytes() == x_after.tobytes()
    ck.close()


# ------------------------------------------------------------------ guard bands


def test_guard_bands_notice_a_single_element_written_outside_a_buffer():
    """The checker itself: a guarded context reports clean bands after a save and a recovery, and reports the
    damage when one element right behind the running checkpoint (inside the allocation's own guard band, so the
    write is harmless) is overwritten."""
    w = make_workload("mf", l_rows=3000, r_rows=100)
    xd = parity.to_dev(w.x)
    ck = api.ScarCheckpoint(xd, n_shards=4, row_elems=w.geom.row_elems, block_elems=w.geom.block_elems, guarded=True)
    ck.load(parity.to_dev(w.z))
    ck.priority_save(0.3)
    ck.recover_partial_blocks(parity.to_dev(w.lost_blocks))
    assert ck.check_guards() == 0
    n = w.x.size
    z_addr = api.scar_ckpt_view(ck.ctx)["z"]
    behind = api.device_array(z_addr + 4 * n, 1, np.float32)  # first element of the band behind z
    before = behind.clone()
    behind.fill_(1.0)
    torch.cuda.synchronize()
    assert ck.check_guards() == 4
    behind.copy_(before)
    torch.cuda.synchronize()
    assert ck.check_guards() == 0
    plain = api.ScarCheckpoint(parity.to_dev(w.x), block_elems=w.geom.block_elems)
    with pytest.raises(api.ScarError) as e:
        plain.check_guards()
    assert e.value.code == -5
    plain.close()
    ck.close()
