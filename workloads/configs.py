"""Seeded generators for the five synthetic parameter sets.

Each generator returns a :class:`Workload`: the running checkpoint ``z``, the
live parameters ``x = z + delta`` (formed in the element type, so every later
definition applies to the stored values), the block geometry and the lost set
used for the recovery leg.  The shapes imitate the paper's four model families
(Section 5.1: MLR weight matrix, MF factor matrices, LDA count table, CNN
weights) plus one tiny vector; the paper's datasets themselves are not used.

Nothing here computes a distance, a ranking, a packed payload or a norm.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np


@dataclass(frozen=True)
class Geometry:
    """Block geometry of a flat parameter buffer.

    ``row_elems == 0`` means a single row of ``n_elems``.  Blocks are
    ``block_elems`` long, never straddle a row, and the last block of a row
    may be shorter.  Shard ``s`` of ``n_shards`` owns the contiguous block
    range ``[floor(s*B/S), floor((s+1)*B/S))``.
    """

    n_elems: int
    row_elems: int
    block_elems: int
    n_shards: int = 8

    @property
    def row_len(self) -> int:
        return self.row_elems if self.row_elems else self.n_elems

    @property
    def n_rows(self) -> int:
        return self.n_elems // self.row_len if self.n_elems else 0

    @property
    def blocks_per_row(self) -> int:
        return -(-self.row_len // self.block_elems) if self.n_elems else 0

    @property
    def n_blocks(self) -> int:
        return self.n_rows * self.blocks_per_row


def block_offsets(geom: Geometry) -> np.ndarray:
    """Element offset of every block plus the end sentinel (``B + 1`` uint64)."""
    if geom.n_elems == 0:
        return np.zeros(1, dtype=np.uint64)
    in_row = np.arange(geom.blocks_per_row, dtype=np.uint64) * np.uint64(geom.block_elems)
    rows = np.arange(geom.n_rows, dtype=np.uint64) * np.uint64(geom.row_len)
    off = (rows[:, None] + in_row[None, :]).reshape(-1)
    return np.concatenate([off, np.array([geom.n_elems], dtype=np.uint64)])


def shard_block_ranges(n_blocks: int, n_shards: int) -> np.ndarray:
    """``(S, 2)`` int64 array of ``[first, last)`` block ids per shard."""
    s = np.arange(n_shards + 1, dtype=object) * n_blocks // n_shards
    s = np.array(s, dtype=np.int64)
    return np.stack([s[:-1], s[1:]], axis=1)


@dataclass
class Workload:
    name: str
    dtype: str  # "f32" or "i32"
    geom: Geometry
    z: np.ndarray  # running checkpoint, flat
    x: np.ndarray  # live parameters, flat
    r_values: Tuple[float, ...]
    lost_shards: Optional[np.ndarray] = None  # uint8[n_shards], 0 alive / 1 lost
    lost_blocks: Optional[np.ndarray] = None  # uint8[n_blocks]
    seed: int = 0
    notes: dict = field(default_factory=dict)

    @property
    def n_blocks(self) -> int:
        return self.geom.n_blocks


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def _lose_shards(rng: np.random.Generator, n_shards: int, n_lost: int) -> np.ndarray:
    mask = np.zeros(n_shards, dtype=np.uint8)
    mask[rng.choice(n_shards, size=n_lost, replace=False)] = 1
    return mask


def make_tiny(n_elems: int = 1 << 20, block_elems: int = 256, seed: int = 0) -> Workload:
    """fp32 vector; per-block Gaussian delta whose scale is LogNormal(0, 1)."""
    rng = _rng(seed)
    geom = Geometry(n_elems, 0, block_elems, 8)
    n_blocks = geom.n_blocks
    z = rng.standard_normal(n_elems, dtype=np.float32)
    sigma = rng.lognormal(0.0, 1.0, size=n_blocks).astype(np.float32)
    lens = np.diff(block_offsets(geom)).astype(np.int64)
    delta = rng.standard_normal(n_elems, dtype=np.float32) * np.repeat(sigma, lens)
    x = (z + delta).astype(np.float32)
    return Workload("tiny", "f32", geom, z, x, (0.25,), lost_shards=_lose_shards(rng, 8, 4), seed=seed)


def make_mlr(rows: int = 1000, cols: int = 100_000, block_elems: int = 1024, seed: int = 1,
             col_frac: float = 0.05) -> Workload:
    """fp32 ``rows x cols`` weight matrix; delta only on a random 5 % of the columns."""
    rng = _rng(seed)
    geom = Geometry(rows * cols, cols, block_elems, 8)
    z = rng.standard_normal(rows * cols, dtype=np.float32) * np.float32(1e-2)
    n_hot = max(1, int(round(col_frac * cols)))
    hot = np.sort(rng.choice(cols, size=n_hot, replace=False))
    x2 = z.reshape(rows, cols).copy()
    d = rng.standard_normal((rows, n_hot), dtype=np.float32) * np.float32(1e-3)
    x2[:, hot] = (x2[:, hot] + d).astype(np.float32)
    x = x2.reshape(-1)
    lost = np.zeros(8, dtype=np.uint8)
    lost[int(rng.integers(8))] = 1
    return Workload("mlr", "f32", geom, z, x, (0.05, 0.25), lost_shards=lost, seed=seed,
                    notes={"hot_columns": hot})


def make_mf(l_rows: int = 480_000, r_rows: int = 18_000, rank: int = 100, seed: int = 2,
            lost_frac: float = 0.25) -> Workload:
    """fp32 factors ``L`` then ``R`` in one buffer, one block per 100-float row.

    Row delta scale follows a Zipf(1.1) "degree" (clipped at 1e4) divided by its
    mean; a random quarter of the ``L`` rows is lost, ``R`` rows never are.
    """
    rng = _rng(seed)
    n_rows = l_rows + r_rows
    geom = Geometry(n_rows * rank, rank, rank, 8)
    z = rng.random(n_rows * rank, dtype=np.float32)
    deg = np.minimum(rng.zipf(1.1, size=n_rows), 10_000).astype(np.float64)
    scale = (deg / deg.mean() * 1e-2).astype(np.float32)
    delta = rng.standard_normal((n_rows, rank), dtype=np.float32) * scale[:, None]
    x = (z.reshape(n_rows, rank) + delta).astype(np.float32).reshape(-1)
    lost = np.zeros(n_rows, dtype=np.uint8)
    lost[rng.choice(l_rows, size=int(round(lost_frac * l_rows)), replace=False)] = 1
    return Workload("mf", "f32", geom, z, x, (0.1,), lost_blocks=lost, seed=seed)


def make_lda(vocab: int = 100_000, topics: int = 1000, seed: int = 3, lam_max: float = 50.0) -> Workload:
    """int32 word-topic count table, one block per word row.

    ``z ~ Poisson(2)``; word ``w`` has rate ``lam_max * rank_w**-1.05`` with
    ``rank`` a seeded permutation; each cell moves by the difference of two
    Poisson draws at that rate and is clamped at zero.
    """
    rng = _rng(seed)
    geom = Geometry(vocab * topics, topics, topics, 8)
    z = rng.poisson(2.0, size=(vocab, topics)).astype(np.int32)
    rank = rng.permutation(vocab).astype(np.float64) + 1.0
    lam = lam_max * rank ** -1.05
    x = np.empty_like(z)
    step = max(1, (1 << 24) // topics)
    for lo in range(0, vocab, step):
        hi = min(vocab, lo + step)
        l2 = np.broadcast_to(lam[lo:hi, None], (hi - lo, topics))
        d = rng.poisson(l2).astype(np.int64) - rng.poisson(l2).astype(np.int64)
        x[lo:hi] = np.maximum(z[lo:hi].astype(np.int64) + d, 0).astype(np.int32)
    return Workload("lda", "i32", geom, z.reshape(-1), x.reshape(-1), (0.2,),
                    lost_shards=_lose_shards(rng, 8, 2), seed=seed)


def make_cnn(n_elems: int = 1 << 30, block_elems: int = 4096, seed: int = 4) -> Workload:
    """fp32 vector; per-block scale ``1 + Pareto(1.5)`` times N(0, 1e-4) noise.

    Host (numpy) form, generated in chunks.  At the full 2**30 elements this
    needs about 8 GiB of host memory for ``x`` and ``z``; the device form
    :func:`make_cnn_device` is the quicker route on a GPU machine.
    """
    rng = _rng(seed)
    geom = Geometry(n_elems, 0, block_elems, 8)
    n_blocks = geom.n_blocks
    a = (1.0 + rng.pareto(1.5, size=n_blocks)).astype(np.float32)
    z = np.empty(n_elems, dtype=np.float32)
    x = np.empty(n_elems, dtype=np.float32)
    chunk_blocks = max(1, (1 << 24) // block_elems)
    for b0 in range(0, n_blocks, chunk_blocks):
        b1 = min(n_blocks, b0 + chunk_blocks)
        lo, hi = b0 * block_elems, min(n_elems, b1 * block_elems)
        zc = rng.standard_normal(hi - lo, dtype=np.float32) * np.float32(5e-2)
        ec = rng.standard_normal(hi - lo, dtype=np.float32) * np.float32(1e-4)
        scale = np.repeat(a[b0:b1], block_elems)[: hi - lo]
        z[lo:hi] = zc
        x[lo:hi] = (zc + scale * ec).astype(np.float32)
    lost = np.zeros(8, dtype=np.uint8)
    lost[int(rng.integers(8))] = 1
    return Workload("cnn", "f32", geom, z, x, (0.01, 0.1, 0.5, 1.0), lost_shards=lost, seed=seed)


def make_cnn_device(n_elems: int = 1 << 30, block_elems: int = 4096, seed: int = 4, device="cuda:0"):
    """Device form of the CNN-scale set: returns ``(geom, z, x, lost_shards)``.

    ``z`` and ``x`` are torch tensors on ``device`` drawn from a seeded torch
    generator, chunk by chunk, with the same recipe as :func:`make_cnn` (the
    bytes differ from the numpy form; a caller that needs host copies takes
    them from these tensors so every consumer sees the same data).
    """
    import torch

    geom = Geometry(n_elems, 0, block_elems, 8)
    n_blocks = geom.n_blocks
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    u = torch.rand(n_blocks, generator=g, device=device, dtype=torch.float32)
    a = (1.0 - u).clamp_min(1e-12).pow(-1.0 / 1.5)
    z = torch.empty(n_elems, device=device, dtype=torch.float32)
    x = torch.empty(n_elems, device=device, dtype=torch.float32)
    chunk_blocks = max(1, (1 << 26) // block_elems)
    for b0 in range(0, n_blocks, chunk_blocks):
        b1 = min(n_blocks, b0 + chunk_blocks)
        lo, hi = b0 * block_elems, min(n_elems, b1 * block_elems)
        zc = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32) * 5e-2
        ec = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32) * 1e-4
        scale = a[b0:b1].repeat_interleave(block_elems)[: hi - lo]
        z[lo:hi] = zc
        x[lo:hi] = zc + scale * ec
    lost = np.zeros(8, dtype=np.uint8)
    lost[int(_rng(seed).integers(8))] = 1
    return geom, z, x, lost


def bylayer_offsets(scale: int = 1, pad_to: int = 1) -> np.ndarray:
    """Block offsets of a network checkpointed by layer (Section 5.1, by-layer partitioning): weight and bias of two
    convolutions and three fully connected layers, each tensor one block, so block lengths span five orders of
    magnitude.  ``scale`` widens every layer; ``pad_to`` rounds lengths up (4 keeps every block 16-byte aligned)."""
    c1, c2, f1, f2, classes = 32 * scale, 64 * scale, 1024 * scale, 512 * scale, 10
    lens = [25 * 1 * c1, c1, 25 * c1 * c2, c2, 49 * c2 * f1, f1, f1 * f2, f2, f2 * classes, classes]
    lens = [-(-n // pad_to) * pad_to for n in lens]
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)


def make_cnn_bylayer(scale: int = 1, pad_to: int = 1, dtype: str = "f32", seed: int = 5):
    """Returns ``(boff, z, x)`` for the by-layer layout: per-layer change scale ``1 + Pareto(1.5)`` times
    N(0, 1e-3) noise around N(0, 5e-2) weights (float32), or Poisson counts with small integer changes (int32)."""
    rng = _rng(seed)
    boff = bylayer_offsets(scale, pad_to)
    lens = np.diff(boff.astype(np.int64))
    n = int(boff[-1])
    if dtype == "f32":
        z = (rng.standard_normal(n, dtype=np.float32) * np.float32(5e-2)).astype(np.float32)
        a = (1.0 + rng.pareto(1.5, size=lens.size)).astype(np.float32)
        x = (z + rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3) * np.repeat(a, lens)).astype(np.float32)
    else:
        z = rng.poisson(3.0, size=n).astype(np.int32)
        x = np.maximum(z + rng.integers(-2, 3, size=n), 0).astype(np.int32)
    return boff, z, x


CONFIGS = {
    "tiny": make_tiny,
    "mlr": make_mlr,
    "mf": make_mf,
    "lda": make_lda,
    "cnn": make_cnn,
}


def make_workload(name: str, **kw) -> Workload:
    """Build one of the five sets by name; keyword arguments shrink or reseed it."""
    return CONFIGS[name](**kw)
