"""The selection run many times in a row on changing inputs (Section 4.3, checkpoint step 3).  The set it must
return has a plain definition, the k blocks with the largest scores, equal scores to the lowest ids, so every
run is checked exactly (ids, offsets, totals) against a stable sort of the scores the library itself computed:
no floating-point freedom is left.  The kernel's CTAs hand work to one another through memory several times per
run, and a mistake in such a protocol shows up once in many runs, not in one; hence hundreds of runs per
grid shape (one CTA; a few; about half the SMs; nearly all; more tiles than SMs), with many exact ties."""

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1810_07354_b200 import api  # noqa: E402


@pytest.mark.parametrize("nb,blk,rows,reps", [
    (4096, 16, 0, 150),      # one CTA, histograms in shared memory
    (3000, 16, 0, 150),      # one CTA, ragged tile
    (20_000, 16, 0, 150),    # five CTAs
    (300_000, 8, 0, 100),    # 74 CTAs
    (0, 1024, 300, 150),     # 300 rows of 100 000 in blocks of 1024 (tail 672): two block lengths, 8 CTAs
    (600_000, 4, 0, 30),     # 147 CTAs
    (700_000, 4, 0, 30),     # more tiles than SMs: several tiles per CTA
])
def test_repeated_selections_are_exact(nb, blk, rows, reps):
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev)
    g.manual_seed(1000 + nb + rows)
    row = 100_000 if rows else 0
    n = rows * row if rows else nb * blk
    z = torch.randn(n, device=dev, generator=g)
    x = z.clone()
    ck = api.ScarCheckpoint(x, n_shards=8, row_elems=row, block_elems=blk)
    nb = ck.n_blocks
    lens = np.tile(np.r_[np.full(97, 1024), 672], rows).astype(np.int64) if rows else np.full(nb, blk, dtype=np.int64)
    d_lens = torch.from_numpy(lens).to(dev)
    ids = np.arange(nb)
    for it in range(reps):
        # a random subset of the blocks moves, by quantised amounts: many exactly equal scores, many exact zeros
        frac = (0.02, 0.3, 0.9)[it % 3]
        moved = (torch.rand(nb, device=dev, generator=g) < frac).float()
        step = torch.randint(0, 4 if it % 2 else 1000, (nb,), device=dev, generator=g).float() * 0.25
        x.copy_(z + torch.repeat_interleave(moved * step, d_lens))
        ck.load(z)
        if it % 5:
            k = int(torch.randint(0, nb + 1, (1,), generator=g, device=dev).item())
        else:
            k = (0, 1, nb - 1, nb, nb // 2)[(it // 5) % 5]
        info = ck.priority_save_k(k)
        v = ck.views(k=k)
        scores = v["scores"].cpu().numpy()
        sel = v["sel"].cpu().numpy().astype(np.int64) & 0xFFFFFFFF
        want = np.sort(np.lexsort((ids, -scores.astype(np.float64)))[:k])
        assert int(info.k) == k
        assert np.array_equal(sel, want), f"run {it}: k={k}"
        offs = np.concatenate([[0], np.cumsum(lens[want])])
        assert np.array_equal(v["poff"].cpu().numpy(), offs), f"run {it}: k={k}"
        assert int(info.payload_elems) == int(offs[-1])
    ck.close()


@pytest.mark.parametrize("rows,row,blk", [(200_000, 100, 100), (4096, 256, 256), (3000, 4096, 4096)])
def test_repeated_norms_give_the_same_bits(rows, row, blk):
    """The reduction that ends a norm pass hands per-CTA sums to a few collecting CTAs through memory (the
    perturbation norm of Theorem 4.1 over a lost set).  Its order of additions depends on the grid alone, so 300
    runs over one input must give one bit pattern, for the whole vector, for lost shards and for a block mask;
    and the count of blocks and elements must be the lost set's every time."""
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev)
    g.manual_seed(rows)
    n = rows * row
    z = torch.randn(n, device=dev, generator=g)
    x = z + 0.01 * torch.randn(n, device=dev, generator=g)
    ck = api.ScarCheckpoint(x, n_shards=8, row_elems=row, block_elems=blk)
    ck.load(z)
    nb = ck.n_blocks
    lost_shards = np.array([0, 1, 0, 0, 1, 1, 0, 1], dtype=np.uint8)
    mask = (torch.rand(nb, device=dev, generator=g) < 0.25).to(torch.uint8)
    n_mask = int(mask.sum().item())
    first = None
    for it in range(300):
        a = ck.perturbation_norm(None)
        b = ck.perturbation_norm(lost_shards)
        c = ck.perturbation_norm_blocks(mask)
        got = (np.float64(a.l2).tobytes(), np.float64(b.l2).tobytes(), np.float64(c.l2).tobytes(),
               int(a.lost_blocks), int(b.lost_blocks), int(c.lost_blocks), int(a.lost_elems), int(c.lost_elems))
        if first is None:
            first = got
            assert int(a.lost_blocks) == nb and int(a.lost_elems) == n
            assert int(c.lost_blocks) == n_mask and int(c.lost_elems) == n_mask * blk
            assert a.l2 > b.l2 > 0 and a.l2 > c.l2 > 0
        assert got == first, f"run {it}"
    ck.close()
