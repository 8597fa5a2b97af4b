"""Pins for the CPU oracle: what the paper and the arithmetic fix, not the oracle's own formulae.

Each test names the passage it checks.  The brute-force forms below are
written independently of ``oracle/`` (explicit per-element block-id arrays,
Python ``sorted`` with a key, exact integer arithmetic).
"""

import json
import math
import os

import numpy as np
import pytest

import oracle
from workloads import Geometry, block_offsets, make_workload, shard_block_ranges


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def ragged_boff(r, n_blocks, max_len=9, allow_empty=True):
    lens = r.integers(0 if allow_empty else 1, max_len + 1, size=n_blocks)
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)


def block_ids(boff):
    """Per-element block id, the independent way of saying which block an element is in."""
    lens = np.diff(boff.astype(np.int64))
    return np.repeat(np.arange(lens.size), lens)


# ---------------------------------------------------------------- hand-worked example


@pytest.fixture(scope="module")
def hand(golden_dir):
    with open(os.path.join(golden_dir, "hand_example.json")) as f:
        return json.load(f)


def test_hand_example_float(hand):
    boff = np.array(hand["boff"], dtype=np.uint64)
    x = np.array(hand["x"], dtype=np.float32)
    z = np.array(hand["z"], dtype=np.float32)
    res = oracle.priority_save(x, z, boff, k=hand["k"])
    assert res.scores.tolist() == hand["scores"]
    assert res.sel.tolist() == hand["sel"]
    assert res.poff.tolist() == hand["poff"]
    assert res.payload.tolist() == hand["payload"]
    assert res.z_after.tolist() == hand["z_after"]
    assert oracle.block_scores(x, res.z_after, boff).tolist() == hand["scores_after"]
    lost = np.array(hand["lost_blocks"], dtype=np.uint8)
    part = oracle.perturbation_norm(x, z, boff, lost)
    assert part.sumsq == hand["partial_sumsq"] and part.l2 == math.sqrt(hand["partial_sumsq"])
    assert (part.lost_blocks, part.lost_elems) == (3, 8)
    assert oracle.perturbation_norm(x, z, boff, None).sumsq == hand["full_sumsq"]
    rec, x_after = oracle.recover_partial(x, z, boff, lost)
    assert rec.sumsq == hand["partial_sumsq"]
    assert x_after.tolist() == hand["x_recovered"]
    assert x.tolist() == hand["x"], "recover_partial must not modify its input"


def test_hand_example_int(hand):
    boff = np.array(hand["boff"], dtype=np.uint64)
    x = np.array(hand["x"], dtype=np.int32)
    z = np.array(hand["z"], dtype=np.int32)
    res = oracle.priority_save(x, z, boff, k=hand["k"])
    assert res.scores.dtype == np.uint64 and res.scores.tolist() == hand["l1_scores"]
    assert res.sel.tolist() == hand["sel"]  # l1 ranks the same two blocks here
    assert res.payload.tolist() == hand["payload"] and res.z_after.tolist() == hand["z_after"]
    lost = np.array(hand["lost_blocks"], dtype=np.uint8)
    assert oracle.perturbation_norm(x, z, boff, lost).l1 == hand["l1_partial"]
    assert oracle.perturbation_norm(x, z, boff, None).l1 == hand["l1_full"]
    _, x_after = oracle.recover_partial(x, z, boff, lost)
    assert x_after.tolist() == hand["x_recovered"]


# ---------------------------------------------------------------- geometry


@pytest.mark.parametrize("n,row,blk", [(0, 0, 4), (10, 0, 4), (12, 0, 4), (30, 10, 4), (30, 10, 10), (30, 10, 16),
                                       (7, 7, 1), (100_000 * 3, 100_000, 1024)])
def test_layout_offsets_match_generator_geometry(n, row, blk):
    boff = oracle.layout_offsets(n, row, blk)
    ref = block_offsets(Geometry(n, row, blk))
    assert boff.tolist() == ref.tolist()
    if n:
        lens = np.diff(boff.astype(np.int64))
        assert lens.min() >= 1 and lens.max() <= blk and lens.sum() == n
        row_len = row or n
        # no block crosses a row end
        assert np.all(boff[:-1].astype(np.int64) // row_len == (boff[1:].astype(np.int64) - 1) // row_len)


def test_mlr_geometry_has_672_tail():
    boff = oracle.layout_offsets(2 * 100_000, 100_000, 1024)
    lens = np.diff(boff.astype(np.int64))
    assert lens.size == 2 * 98 and lens[97] == 672 and lens[98] == 1024 and lens[-1] == 672


@pytest.mark.parametrize("nb,ns", [(16, 8), (10, 3), (3, 8), (0, 4), (98_000, 8), (1, 1), (7, 7)])
def test_expand_shards_is_a_partition(nb, ns):
    ranges = shard_block_ranges(nb, ns)
    total = np.zeros(nb, dtype=np.int64)
    for s in range(ns):
        m = np.zeros(ns, dtype=np.uint8)
        m[s] = 7  # any non-zero byte means lost
        e = oracle.expand_shards(nb, m)
        assert set(np.unique(e).tolist()) <= {0, 1}
        lo, hi = ranges[s]
        ref = np.zeros(nb, dtype=np.uint8)
        ref[lo:hi] = 1
        assert e.tolist() == ref.tolist()
        total += e
    assert np.all(total == 1), "every block belongs to exactly one shard"
    assert oracle.expand_shards(nb, np.zeros(ns, np.uint8)).sum() == 0
    assert oracle.expand_shards(nb, np.ones(ns, np.uint8)).sum() == nb


# ---------------------------------------------------------------- scores (checkpoint step 1)


def test_scores_zero_right_after_init():
    # Section 4.2: the running checkpoint starts at x^(0), so nothing has changed yet.
    w = make_workload("tiny", n_elems=1 << 12)
    z = oracle.ckpt_init(w.x)
    assert z is not w.x and z.tobytes() == w.x.tobytes()
    s = oracle.block_scores(w.x, z, block_offsets(w.geom))
    assert s.dtype == np.float64 and np.all(s == 0.0)


def test_score_of_a_single_power_of_two_change_is_exact():
    boff = oracle.layout_offsets(40, 20, 8)  # lengths 8, 8, 4, 8, 8, 4
    z = rng(5).standard_normal(40).astype(np.float32)
    for pos, blk in [(0, 0), (7, 0), (8, 1), (19, 2), (20, 3), (39, 5)]:
        x = z.copy()
        x[pos] = np.float32(2.0)  # pick z so that the difference is exactly 2^-3
        z2 = z.copy()
        z2[pos] = np.float32(2.0 - 0.125)
        s = oracle.block_scores(x, z2, boff)
        want = np.zeros(6)
        want[blk] = 2.0 ** -6
        assert s.tolist() == want.tolist()
        # the score is symmetric in x and z (a squared distance)
        assert oracle.block_scores(z2, x, boff).tolist() == want.tolist()


def test_scores_match_bruteforce_exactly_on_integer_valued_floats():
    r = rng(11)
    boff = ragged_boff(r, 200)
    n = int(boff[-1])
    x = r.integers(-50, 50, size=n).astype(np.float32)
    z = r.integers(-50, 50, size=n).astype(np.float32)
    want = np.zeros(200, dtype=np.int64)
    np.add.at(want, block_ids(boff), (x.astype(np.int64) - z.astype(np.int64)) ** 2)
    got = oracle.block_scores(x, z, boff)
    assert got.tolist() == want.astype(np.float64).tolist()
    assert np.all(got[np.diff(boff.astype(np.int64)) == 0] == 0.0), "empty blocks score 0"


def test_scores_match_fsum_on_random_floats():
    r = rng(12)
    boff = ragged_boff(r, 64, max_len=40)
    n = int(boff[-1])
    x = r.standard_normal(n).astype(np.float32)
    z = (x + r.standard_normal(n).astype(np.float32) * np.float32(1e-3)).astype(np.float32)
    got = oracle.block_scores(x, z, boff)
    for b in range(64):
        lo, hi = int(boff[b]), int(boff[b + 1])
        exact = math.fsum((float(x[i]) - float(z[i])) ** 2 for i in range(lo, hi))
        assert got[b] == pytest.approx(exact, rel=1e-13, abs=0.0)


def test_scores_use_the_stored_float32_values_not_wider_ones():
    # x is formed in float32; the definition applies to the stored values.
    z = np.array([1.0], dtype=np.float32)
    x = np.array([1.0 + 2.0 ** -30], dtype=np.float32)  # rounds back to 1.0 in float32
    assert oracle.block_scores(x, z, np.array([0, 1], dtype=np.uint64))[0] == 0.0


def test_int_scores_exact_including_extremes():
    boff = np.array([0, 2, 3, 6], dtype=np.uint64)
    imax, imin = np.iinfo(np.int32).max, np.iinfo(np.int32).min
    x = np.array([imax, imin, 5, -3, 0, 9], dtype=np.int32)
    z = np.array([imin, imax, 5, 4, -1, 2], dtype=np.int32)
    s = oracle.block_scores(x, z, boff)
    assert s.dtype == np.uint64
    assert s.tolist() == [2 * (2 ** 32 - 1), 0, 7 + 1 + 7]
    assert oracle.perturbation_norm(x, z, boff).l1 == 2 * (2 ** 32 - 1) + 15


def test_int_scores_match_python_integers():
    r = rng(13)
    boff = ragged_boff(r, 100)
    n = int(boff[-1])
    x = r.integers(-2 ** 31, 2 ** 31, size=n).astype(np.int32)
    z = r.integers(-2 ** 31, 2 ** 31, size=n).astype(np.int32)
    got = oracle.block_scores(x, z, boff).tolist()
    ids = block_ids(boff)
    want = [0] * 100
    for i in range(n):
        want[ids[i]] += abs(int(x[i]) - int(z[i]))
    assert got == want


def test_lda_l1_is_twice_length_scaled_total_variation():
    # Appendix C: total variation of a document's topic distribution, scaled by its length.
    # For two count rows with the same total L: L * TV(n/L, m/L) = (1/2) * sum |n - m|.
    r = rng(14)
    topics, length = 20, 500
    n = r.multinomial(length, np.full(topics, 1 / topics)).astype(np.int32)
    m = r.multinomial(length, np.full(topics, 1 / topics)).astype(np.int32)
    tv = 0.5 * np.abs(n / length - m / length).sum()
    got = oracle.block_scores(n, m, np.array([0, topics], dtype=np.uint64))[0]
    assert int(got) == pytest.approx(2 * length * tv, rel=1e-12)


# ---------------------------------------------------------------- k from r


def test_k_table(golden_dir):
    rows = 0
    with open(os.path.join(golden_dir, "k_table.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            r, nb, k = line.split()
            assert oracle.k_from_r(float(r), int(nb)) == int(k), line
            rows += 1
    assert rows >= 20


@pytest.mark.parametrize("bad", [-0.1, 1.0000001, float("nan"), float("inf"), -float("inf")])
def test_k_rejects_r_outside_unit_interval(bad):
    with pytest.raises(ValueError):
        oracle.k_from_r(bad, 100)


def test_k_is_monotone_in_r():
    ks = [oracle.k_from_r(r, 997) for r in np.linspace(0, 1, 2001)]
    assert ks[0] == 0 and ks[-1] == 997 and all(a <= b for a, b in zip(ks, ks[1:]))


# ---------------------------------------------------------------- selection (checkpoint step 3)


def brute_top_k(score, k):
    key = [math.inf if (isinstance(s, float) and (math.isnan(s) or math.isinf(s))) else s for s in score]
    order = sorted(range(len(key)), key=lambda b: (-key[b], b))
    return sorted(order[:k])


@pytest.mark.parametrize("seed", range(6))
def test_selection_matches_bruteforce_sort_with_many_ties(seed):
    r = rng(100 + seed)
    nb = int(r.integers(1, 300))
    score = r.integers(0, 6, size=nb).astype(np.float64)  # few distinct values: ties everywhere
    for k in sorted({0, 1, nb // 3, nb - 1, nb} & set(range(nb + 1))):
        sel, bad = oracle.select_top_k(score, k)
        assert bad == 0 and sel.dtype == np.uint32
        assert sel.tolist() == brute_top_k(score.tolist(), k)
    su = score.astype(np.uint64)
    for k in (0, nb // 2, nb):
        assert oracle.select_top_k(su, k)[0].tolist() == brute_top_k(su.tolist(), k)


def test_selection_special_orders():
    nb, k = 50, 7
    assert oracle.select_top_k(np.full(nb, 3.5), k)[0].tolist() == list(range(k)), "all equal: lowest ids"
    assert oracle.select_top_k(np.zeros(nb), k)[0].tolist() == list(range(k)), "exact-zero ties: lowest ids"
    inc = np.arange(nb, dtype=np.float64)
    assert oracle.select_top_k(inc, k)[0].tolist() == list(range(nb - k, nb)), "increasing: the last k"
    assert oracle.select_top_k(inc[::-1].copy(), k)[0].tolist() == list(range(k)), "decreasing: the first k"
    big = np.array([2 ** 63, 5, 2 ** 63 + 1, 2 ** 64 - 1, 0], dtype=np.uint64)
    assert oracle.select_top_k(big, 2)[0].tolist() == [2, 3], "uint64 scores compare as unsigned 64-bit"


def test_selection_nonfinite_scores_rank_first():
    score = np.array([1.0, np.nan, 5.0, np.inf, 2.0, np.nan])
    sel, bad = oracle.select_top_k(score, 2)
    assert bad == 3 and sel.tolist() == [1, 3]  # all three rank as +inf, ties to the lowest ids
    sel, _ = oracle.select_top_k(score, 4)
    assert sel.tolist() == [1, 2, 3, 5]


def test_priority_set_minimises_the_residual():
    # Section 4.2: saving what changed most is what shrinks the perturbation a failure would cause.
    # For additive block scores the top-k set leaves the least unsaved change of all size-k sets.
    r = rng(21)
    nb, k = 400, 50
    score = r.lognormal(0, 1.5, size=nb)
    sel, _ = oracle.select_top_k(score, k)
    best = score.sum() - score[sel].sum()
    for _ in range(1000):
        other = r.choice(nb, size=k, replace=False)
        assert best <= score.sum() - score[other].sum() + 1e-9
    for start in range(0, nb, 37):  # round-robin windows (Section 5.4's "round" strategy)
        rr = (start + np.arange(k)) % nb
        assert best <= score.sum() - score[rr].sum() + 1e-9


# ---------------------------------------------------------------- pack / update (checkpoint step 4)


def small_case(seed, dtype=np.float32, nb=60):
    r = rng(seed)
    boff = ragged_boff(r, nb, allow_empty=False)
    n = int(boff[-1])
    if dtype == np.float32:
        z = r.standard_normal(n).astype(np.float32)
        x = (z + r.standard_normal(n).astype(np.float32) * np.repeat(r.lognormal(0, 1, nb), np.diff(boff.astype(np.int64))).astype(np.float32)).astype(np.float32)
    else:
        z = r.poisson(2.0, size=n).astype(np.int32)
        x = np.maximum(z + r.integers(-3, 4, size=n), 0).astype(np.int32)
    return x, z, boff


@pytest.mark.parametrize("dtype", [np.float32, np.int32])
def test_r_equal_one_is_a_full_checkpoint(dtype):
    # Section 4: the traditional checkpoint saves the whole state.
    x, z, boff = small_case(31, dtype)
    res = oracle.priority_save(x, z, boff, r=1.0)
    nb = boff.size - 1
    assert res.k == nb and res.sel.tolist() == list(range(nb))
    assert res.payload.tobytes() == x.tobytes()
    assert res.z_after.tobytes() == x.tobytes()
    assert res.poff.tolist() == boff.tolist()
    assert not np.any(oracle.block_scores(x, res.z_after, boff))
    assert z.tobytes() != x.tobytes(), "inputs are not modified"


@pytest.mark.parametrize("dtype", [np.float32, np.int32])
def test_k_zero_changes_nothing(dtype):
    x, z, boff = small_case(32, dtype)
    res = oracle.priority_save(x, z, boff, r=0.0)
    assert res.k == 0 and res.sel.size == 0 and res.payload.size == 0 and res.poff.tolist() == [0]
    assert res.z_after.tobytes() == z.tobytes()


@pytest.mark.parametrize("dtype", [np.float32, np.int32])
def test_partial_save_bytes_and_residual_identity(dtype):
    x, z, boff = small_case(33, dtype)
    nb = boff.size - 1
    res = oracle.priority_save(x, z, boff, r=0.3)
    ids = block_ids(boff)
    chosen = np.isin(ids, res.sel)
    # payload is x restricted to the chosen blocks, in ascending element order
    assert res.payload.tobytes() == x[chosen].tobytes()
    lens = np.diff(boff.astype(np.int64))
    assert res.poff.tolist() == np.concatenate([[0], np.cumsum(lens[res.sel])]).tolist()
    # the cache takes x on chosen blocks and keeps z elsewhere
    assert res.z_after[chosen].tobytes() == x[chosen].tobytes()
    assert res.z_after[~chosen].tobytes() == z[~chosen].tobytes()
    after = oracle.block_scores(x, res.z_after, boff)
    assert not np.any(after[res.sel])
    unsel = np.setdiff1d(np.arange(nb), res.sel)
    assert after[unsel].tolist() == res.scores[unsel].tolist()
    # what is left unsaved is the total minus what was saved
    if dtype == np.float32:
        total = oracle.perturbation_norm(x, z, boff).sumsq
        left = oracle.perturbation_norm(x, res.z_after, boff).sumsq
        assert left == pytest.approx(total - res.scores[res.sel].sum(), rel=1e-12)
    else:
        total = oracle.perturbation_norm(x, z, boff).l1
        left = oracle.perturbation_norm(x, res.z_after, boff).l1
        assert left == total - int(res.scores[res.sel].sum())


def test_second_save_takes_remaining_changed_blocks_then_lowest_ids():
    x, z, boff = small_case(34)
    nb = boff.size - 1
    k = nb // 2 + 5
    first = oracle.priority_save(x, z, boff, k=k)
    second = oracle.priority_save(x, first.z_after, boff, k=k)
    remaining = np.setdiff1d(np.arange(nb), first.sel)  # the only blocks with a non-zero score now
    zero_fill = first.sel[: k - remaining.size]  # exact-zero ties go to the lowest ids
    assert second.sel.tolist() == sorted(remaining.tolist() + zero_fill.tolist())
    assert second.z_after.tobytes() == x.tobytes()


def test_nan_payload_survives_bit_exactly():
    boff = np.array([0, 2, 4, 6], dtype=np.uint64)
    z = np.zeros(6, dtype=np.float32)
    x = np.zeros(6, dtype=np.float32)
    x.view(np.uint32)[2] = 0x7FC00123  # a NaN with a payload
    x[4] = 3.0
    res = oracle.priority_save(x, z, boff, k=1)
    assert res.nonfinite_blocks == 1 and res.sel.tolist() == [1]
    assert res.payload.view(np.uint32).tolist() == [0x7FC00123, 0]
    assert res.z_after.view(np.uint32)[2] == 0x7FC00123


# ---------------------------------------------------------------- recovery


@pytest.mark.parametrize("dtype", [np.float32, np.int32])
def test_empty_full_and_repeated_recovery(dtype):
    x, z, boff = small_case(41, dtype)
    nb = boff.size - 1
    none = np.zeros(nb, dtype=np.uint8)
    res, xa = oracle.recover_partial(x, z, boff, none)
    assert (res.l2, res.l1, res.lost_blocks, res.lost_elems) == (0.0, 0, 0, 0) and xa.tobytes() == x.tobytes()
    every = np.ones(nb, dtype=np.uint8)
    res, xa = oracle.recover_partial(x, z, boff, every)
    assert xa.tobytes() == z.tobytes() and res.lost_blocks == nb and res.lost_elems == x.size
    # Example 2.3: full recovery perturbs by x^(T) - x^(C)
    if dtype == np.float32:
        want = math.sqrt(math.fsum((float(a) - float(b)) ** 2 for a, b in zip(x, z)))
        assert res.l2 == pytest.approx(want, rel=1e-13)
        assert oracle.perturbation_norm(x, z, boff, None).l2 == res.l2
    else:
        assert res.l1 == sum(abs(int(a) - int(b)) for a, b in zip(x, z))
        assert oracle.perturbation_norm(x, z, boff, None).l1 == res.l1
    again, xb = oracle.recover_partial(xa, z, boff, every)
    assert (again.l2, again.l1) == (0.0, 0) and xb.tobytes() == xa.tobytes()


def test_recovery_right_after_init_is_free():
    w = make_workload("tiny", n_elems=1 << 12)
    boff = block_offsets(w.geom)
    z = oracle.ckpt_init(w.x)
    lost = oracle.expand_shards(w.n_blocks, w.lost_shards)
    res, xa = oracle.recover_partial(w.x, z, boff, lost)
    assert res.l2 == 0.0 and xa.tobytes() == w.x.tobytes() and res.lost_blocks == w.n_blocks // 2


@pytest.mark.parametrize("dtype", [np.float32, np.int32])
def test_partial_recovery_touches_only_the_lost_blocks(dtype):
    # Appendix proof of Theorem 4.1: x on the complement of S is unchanged by failure and recovery.
    x, z, boff = small_case(42, dtype)
    nb = boff.size - 1
    lost = (rng(43).random(nb) < 0.4).astype(np.uint8)
    res, xa = oracle.recover_partial(x, z, boff, lost)
    in_lost = lost[block_ids(boff)].astype(bool)
    assert xa[in_lost].tobytes() == z[in_lost].tobytes()
    assert xa[~in_lost].tobytes() == x[~in_lost].tobytes()
    assert res.lost_blocks == int(lost.sum()) and res.lost_elems == int(in_lost.sum())
    # the read-only norm reports the same perturbation and writes nothing
    x_copy = x.copy()
    ro = oracle.perturbation_norm(x, z, boff, lost)
    assert (ro.l2, ro.l1) == (res.l2, res.l1) and x.tobytes() == x_copy.tobytes()
    # the perturbation is the sum of the lost blocks' checkpoint scores
    s = oracle.block_scores(x, z, boff)
    if dtype == np.float32:
        assert res.sumsq == pytest.approx(s[lost.astype(bool)].sum(), rel=1e-12)
    else:
        assert res.l1 == int(s[lost.astype(bool)].sum())


def test_theorem_4_1_partial_never_exceeds_full():
    x, z, boff = small_case(44, nb=120)
    nb = boff.size - 1
    full = oracle.perturbation_norm(x, z, boff, None).l2
    r = rng(45)
    for p in (0.0, 0.1, 0.5, 0.9, 1.0):
        for _ in range(20):
            lost = (r.random(nb) < p).astype(np.uint8)
            assert oracle.perturbation_norm(x, z, boff, lost).l2 <= full
    # equality is reached when the surviving blocks carry no change (the proof concludes "<=")
    z2 = z.copy()
    keep = np.zeros(nb, dtype=np.uint8)
    keep[: nb // 2] = 1
    alive = ~keep[block_ids(boff)].astype(bool)
    z2[alive] = x[alive]
    assert oracle.perturbation_norm(x, z2, boff, keep).l2 == oracle.perturbation_norm(x, z2, boff, None).l2


def test_theorem_4_2_partition_identity_and_expectation():
    # Proof of Theorem 4.2: ||delta'||^2 is the sum of (z_i - x_i)^2 over the lost indices, so over
    # any partition into shards the shard perturbations add up to ||delta||^2, and a uniformly
    # random lost fraction p gives p * ||delta||^2 on average.
    w = make_workload("tiny", n_elems=1 << 14)
    boff = block_offsets(w.geom)
    nb = w.n_blocks
    full = oracle.perturbation_norm(w.x, w.z, boff, None).sumsq
    parts = 0.0
    for s in range(8):
        m = np.zeros(8, dtype=np.uint8)
        m[s] = 1
        parts += oracle.perturbation_norm(w.x, w.z, boff, oracle.expand_shards(nb, m)).sumsq
    assert parts == pytest.approx(full, rel=1e-12)
    r = rng(46)
    p, trials = 0.25, 1500
    vals = np.array([oracle.perturbation_norm(w.x, w.z, boff, (r.random(nb) < p).astype(np.uint8)).sumsq
                     for _ in range(trials)])
    stderr = vals.std(ddof=1) / math.sqrt(trials)
    assert abs(vals.mean() - p * full) < 4 * stderr
    assert stderr < 0.05 * p * full, "the check has power"


# ---- weighted norms and total variation (Appendix C) -------------------------------------------


def test_l1_scores_of_distributions_are_twice_the_total_variation():
    """TV(p, q) = max over events A of |p(A) - q(A)| (brute force over all subsets) = (1/2) sum |p - q|."""
    r = rng(40)
    k, nb = 7, 12
    p = r.dirichlet(np.ones(k), size=nb).astype(np.float32)
    q = r.dirichlet(np.ones(k), size=nb).astype(np.float32)
    boff = (np.arange(nb + 1, dtype=np.uint64) * k)
    l1 = oracle.block_scores_norm(p.ravel(), q.ravel(), boff, "l1")
    for b in range(nb):
        d = p[b].astype(np.float64) - q[b].astype(np.float64)
        tv = max(abs(sum(d[i] for i in range(k) if mask >> i & 1)) for mask in range(1 << k))
        # float32 rows do not sum to exactly 1; the two sides differ by at most half that defect
        assert abs(0.5 * l1[b] - tv) <= 0.5 * abs(d.sum()) + 1e-15


def test_length_scaled_tv_of_count_rows_is_half_their_l1():
    """Appendix C: scaling the total variation of a document's topic distribution by the document's length removes
    the bias towards short documents: moving one token costs the same in every document."""
    r = rng(41)
    k = 20
    lengths = np.array([5, 50, 500, 5000])
    counts = np.stack([r.multinomial(n, np.ones(k) / k) for n in lengths])
    moved = counts.copy()
    for d in range(lengths.size):  # re-sample one token: one count down, another up
        src = int(np.flatnonzero(moved[d])[0])
        moved[d, src] -= 1
        moved[d, (src + 1) % k] += 1
    p = (counts / lengths[:, None]).astype(np.float32).ravel()
    q = (moved / lengths[:, None]).astype(np.float32).ravel()
    boff = (np.arange(lengths.size + 1, dtype=np.uint64) * k)
    plain = 0.5 * oracle.block_scores_norm(p, q, boff, "l1")
    scaled = oracle.block_scores_norm(p, q, boff, "l1", weights=lengths / 2.0)
    assert plain[0] > 100 * plain[3]  # unweighted: the short document dominates
    np.testing.assert_allclose(scaled, 1.0, rtol=1e-5)  # scaled: one token each
    # and it equals half the l1 of the count rows themselves (the integer path)
    ints = oracle.block_scores(counts.astype(np.int32).ravel(), moved.astype(np.int32).ravel(), boff)
    np.testing.assert_allclose(scaled, ints / 2.0, rtol=1e-5)


def test_weighted_scores_bruteforce_and_special_weights():
    x, z, boff = small_case(42, np.float32, nb=40)
    nb = boff.size - 1
    ids = block_ids(boff)
    w = rng(43).uniform(0, 3, nb)
    for norm in ("l2", "l1"):
        got = oracle.block_scores_norm(x, z, boff, norm, w)
        for b in range(nb):
            d = x[ids == b].astype(np.float64) - z[ids == b].astype(np.float64)
            want = w[b] * (math.fsum(d * d) if norm == "l2" else math.fsum(np.abs(d)))
            assert math.isclose(got[b], want, rel_tol=1e-13, abs_tol=0.0) or got[b] == want == 0.0
        np.testing.assert_array_equal(oracle.block_scores_norm(x, z, boff, norm, np.ones(nb)),
                                      oracle.block_scores_norm(x, z, boff, norm))
        assert not oracle.block_scores_norm(x, z, boff, norm, np.zeros(nb)).any()
    np.testing.assert_array_equal(oracle.block_scores_norm(x, z, boff, "l2"), oracle.block_scores(x, z, boff))


def test_weighted_perturbation_is_a_norm_and_matches_the_plain_one():
    x, z, boff = small_case(44, np.float32, nb=50)
    nb = boff.size - 1
    r = rng(45)
    w = r.uniform(0.1, 4, nb)
    lost = (r.random(nb) < 0.4).astype(np.uint8)
    plain = oracle.perturbation_norm(x, z, boff, lost)
    same = oracle.perturbation_norm_weighted(x, z, boff, lost, "l2")
    assert math.isclose(same.l2, plain.l2, rel_tol=1e-13) and same.lost_blocks == plain.lost_blocks
    assert same.lost_elems == plain.lost_elems
    for norm in ("l2", "l1"):
        full = oracle.perturbation_norm_weighted(x, z, boff, None, norm, w).l2
        part = oracle.perturbation_norm_weighted(x, z, boff, lost, norm, w).l2
        assert 0 < part <= full  # Theorem 4.1 carries over: disjoint supports
        # homogeneity: scaling the difference by 3 scales the norm by 3
        x3 = (z.astype(np.float64) + 3.0 * (x.astype(np.float64) - z.astype(np.float64)))
        d1 = oracle.block_scores_norm(x, z, boff, norm, w)
        # triangle inequality on random splits of the difference: ||a + b|| <= ||a|| + ||b||
        a = (r.random(x.size) * (x - z)).astype(np.float32)
        b = ((x - z) - a).astype(np.float32)
        zero = np.zeros_like(x)
        na = oracle.perturbation_norm_weighted(a, zero, boff, None, norm, w).l2
        nb_ = oracle.perturbation_norm_weighted(b, zero, boff, None, norm, w).l2
        nab = oracle.perturbation_norm_weighted((a + b).astype(np.float32), zero, boff, None, norm, w).l2
        assert nab <= (na + nb_) * (1 + 1e-12)
        n3 = oracle.perturbation_norm_weighted((3 * (a + b)).astype(np.float32), zero, boff, None, norm, w).l2
        assert math.isclose(n3, 3 * nab, rel_tol=1e-6)
        del x3, d1


def test_weights_change_what_a_prioritized_save_takes():
    # one heavily weighted block with a small change outranks unweighted blocks with larger changes
    nb, blk = 8, 4
    z = np.zeros(nb * blk, dtype=np.float32)
    x = z.copy()
    x[0:4] = 0.1      # block 0: small change
    x[4:8] = 1.0      # block 1: large change
    x[8:12] = 0.5     # block 2
    boff = (np.arange(nb + 1, dtype=np.uint64) * blk)
    assert oracle.save_norm(x, z, boff, 1, "l1").sel.tolist() == [1]
    w = np.ones(nb)
    w[0] = 100.0
    assert oracle.save_norm(x, z, boff, 1, "l1", w).sel.tolist() == [0]
    assert oracle.save_norm(x, z, boff, 2, "l2", w).sel.tolist() == [0, 1]  # 100 * 0.04 = 4 > 4 * 0.25 = 1


# ---- baseline selectors (Section 5.4) ---------------------------------------------------


def test_round_robin_hand_cases():
    sel, nxt = oracle.select_round(10, 4, 8)  # blocks 8, 9, 0, 1
    assert sel.tolist() == [0, 1, 8, 9] and nxt == 2
    sel, nxt = oracle.select_round(10, 4, 2)
    assert sel.tolist() == [2, 3, 4, 5] and nxt == 6
    sel, nxt = oracle.select_round(10, 10, 7)  # a full checkpoint leaves the cursor where it was
    assert sel.tolist() == list(range(10)) and nxt == 7
    sel, nxt = oracle.select_round(10, 0, 3)
    assert sel.size == 0 and nxt == 3
    sel, nxt = oracle.select_round(5, 5, 0)
    assert sel.tolist() == [0, 1, 2, 3, 4] and nxt == 0


@pytest.mark.parametrize("nb,k", [(97, 13), (64, 8), (10, 3), (7, 7), (1000, 1)])
def test_round_robin_covers_every_block_once_per_cycle(nb, k):
    # ceil(B/k) consecutive saves touch every block; before the wrap the selections are disjoint
    cur, seen = 0, np.zeros(nb, dtype=np.int64)
    for i in range(-(-nb // k)):
        sel, cur = oracle.select_round(nb, k, cur)
        assert sel.size == k and np.all(np.diff(sel.astype(np.int64)) > 0)
        seen[sel] += 1
    assert seen.min() >= 1 and seen.sum() == k * (-(-nb // k))
    assert seen.max() <= 2 and (seen == 2).sum() == k * (-(-nb // k)) - nb
    assert cur == (k * (-(-nb // k))) % nb


@pytest.mark.parametrize("seed", range(4))
def test_random_selector_matches_bruteforce_sort(seed):
    r = rng(100 + seed)
    nb = 500
    pri = r.integers(0, 40 if seed % 2 else 2**32, size=nb, dtype=np.uint64).astype(np.uint32)  # odd seeds: many ties
    for k in (0, 1, 17, 250, 499, 500):
        want = sorted(sorted(range(nb), key=lambda b: (-int(pri[b]), b))[:k])
        assert oracle.select_random(pri, k).tolist() == want
    assert oracle.select_random(np.full(nb, 7, dtype=np.uint32), 9).tolist() == list(range(9))
    assert oracle.select_random(np.array([0, 2**32 - 1, 5], dtype=np.uint32), 1).tolist() == [1]


def test_random_selector_is_uniform_when_the_priorities_are():
    # inclusion frequency of every block is k/B when the priorities are iid uniform
    r = rng(7)
    nb, k, trials = 40, 10, 4000
    hits = np.zeros(nb)
    for _ in range(trials):
        hits[oracle.select_random(r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32), k)] += 1
    p = k / nb
    se = math.sqrt(p * (1 - p) / trials)
    assert np.all(np.abs(hits / trials - p) < 4.5 * se)


@pytest.mark.parametrize("dtype", [np.float32, np.int32])
def test_baseline_saves_move_exactly_the_chosen_blocks(dtype):
    x, z, boff = small_case(11, dtype)
    nb = boff.size - 1
    ids = block_ids(boff)
    sel, _ = oracle.select_round(nb, 23, nb - 5)
    res = oracle.save_selected(x, z, boff, sel)
    chosen = np.isin(ids, sel)
    assert res.payload.tobytes() == x[chosen].tobytes()
    assert res.z_after[chosen].tobytes() == x[chosen].tobytes()
    assert res.z_after[~chosen].tobytes() == z[~chosen].tobytes()
    lens = (boff[1:] - boff[:-1])[sel.astype(np.int64)]
    assert res.poff.tolist() == np.concatenate([[0], np.cumsum(lens)]).tolist()
    # a round-robin cycle of full coverage ends in a full checkpoint
    cur, zz = 0, z.copy()
    for _ in range(-(-nb // 7)):
        sel, cur = oracle.select_round(nb, 7, cur)
        zz = oracle.save_selected(x, zz, boff, sel).z_after
    assert zz.tobytes() == x.tobytes()


def test_priority_beats_round_and_random_on_the_residual():
    # Section 4.2's heuristic: for the same k the prioritized save leaves the smallest ||x - z||
    x, z, boff = small_case(12, np.float32, nb=80)
    nb = boff.size - 1
    k = 20
    full = oracle.perturbation_norm(x, z, boff).sumsq
    pri = oracle.priority_save(x, z, boff, k=k)
    best = oracle.perturbation_norm(x, pri.z_after, boff).sumsq
    r = rng(13)
    for trial in range(50):
        sel, _ = oracle.select_round(nb, k, int(r.integers(0, nb)))
        other = oracle.perturbation_norm(x, oracle.save_selected(x, z, boff, sel).z_after, boff).sumsq
        assert best <= other * (1 + 1e-12) <= full * (1 + 1e-12)
        sel = oracle.select_random(r.integers(0, 2**32, size=nb, dtype=np.uint64).astype(np.uint32), k)
        other = oracle.perturbation_norm(x, oracle.save_selected(x, z, boff, sel).z_after, boff).sumsq
        assert best <= other * (1 + 1e-12)


def test_workload_recipes_have_the_stated_structure():
    w = make_workload("mlr", rows=16, cols=5000, seed=1)
    boff = block_offsets(w.geom)
    s = oracle.block_scores(w.x, w.z, boff)
    changed = (w.x != w.z).reshape(16, 5000)
    assert changed.any(axis=0).sum() == 250, "5 % of the columns move"
    assert np.all(changed.any(axis=0) == changed.all(axis=0)) or changed.sum() > 0.99 * 16 * 250
    assert np.count_nonzero(s) > 0
    wl = make_workload("lda", vocab=400, topics=50, seed=3)
    assert wl.x.dtype == np.int32 and wl.x.min() >= 0
    assert oracle.block_scores(wl.x, wl.z, block_offsets(wl.geom)).dtype == np.uint64
    wm = make_workload("mf", l_rows=960, r_rows=36, seed=2)
    assert wm.lost_blocks.sum() == 240 and wm.lost_blocks[960:].sum() == 0


# ------------------------------------------------------------------ the OpenMP build (timing only)


def test_openmp_build_of_the_oracle_agrees_with_the_plain_build():
    """The all-core CPU baseline times the same source compiled with -fopenmp.  Integer results, ids, payload
    bytes and restored buffers must be bit-identical to the plain build's, per-block float scores too (each block
    is still summed in element order by one thread); only the recovery's sum across blocks changes its order."""
    import oracle as ora

    r = np.random.Generator(np.random.PCG64(77))
    nb = 3000
    lens = r.integers(0, 200, size=nb)
    boff = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    n = int(boff[-1])
    lost = (r.random(nb) < 0.4).astype(np.uint8)
    cases = []
    zf = r.standard_normal(n).astype(np.float32)
    cases.append((zf + r.standard_normal(n).astype(np.float32) * np.float32(0.1), zf))
    zi = r.integers(-1000, 1000, size=n).astype(np.int32)
    cases.append(((zi + r.integers(-5, 6, size=n)).astype(np.int32), zi))
    got = {}
    try:
        for omp in (False, True):
            threads = ora.use_openmp(omp)
            assert threads >= 1 and (omp or threads == 1)
            got[omp] = [(ora.priority_save(x, z, boff, k=700), ora.perturbation_norm(x, z, boff, lost),
                         ora.recover_partial(x, z, boff, lost)) for x, z in cases]
    finally:
        ora.use_openmp(False)
    for (s0, n0, (r0, x0)), (s1, n1, (r1, x1)) in zip(got[False], got[True]):
        assert s0.scores.tobytes() == s1.scores.tobytes() and s0.sel.tobytes() == s1.sel.tobytes()
        assert s0.payload.tobytes() == s1.payload.tobytes() and s0.poff.tobytes() == s1.poff.tobytes()
        assert s0.z_after.tobytes() == s1.z_after.tobytes() and x0.tobytes() == x1.tobytes()
        assert (n0.l1, n0.lost_blocks, n0.lost_elems) == (n1.l1, n1.lost_blocks, n1.lost_elems)
        assert abs(n0.sumsq - n1.sumsq) <= 1e-13 * max(n0.sumsq, 1e-300) and abs(r0.l2 - r1.l2) <= 1e-13 * max(r0.l2, 1e-300)
