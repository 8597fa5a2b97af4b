"""The checkpoint protocol of Section 4.3 over several GPUs, one process per GPU.

The paper's nodes each hold a partition of the parameters; a checkpoint has every node compute the distances
of its own parameters (step 1), ship them to a coordinator (step 2), which selects the fraction r with the
largest distances over ALL nodes (step 3), after which every node refreshes its cache and saves the selected
parameters it owns (step 4).  Here a rank owns a contiguous range of the global blocks (the rule shards use),
the exchange is one all-gather of the per-rank score arrays over ``torch.distributed`` (NCCL on GPUs; the arrays
hold 4 or 8 bytes per block), and every rank runs the same deterministic selection on the gathered scores
(``scar_ckpt_priority_save_sharded``), so no coordinator is needed and payloads never leave their GPU.
Recovery needs nothing from here: whichever rank owns lost blocks calls ``recover_partial`` on its own context.

Only bookkeeping lives in this module (ranges, padding of the gather); every step of the path runs in the
library's kernels.
"""

from __future__ import annotations

from typing import Optional, Tuple

from . import api


def rank_block_range(n_global_blocks: int, world: int, rank: int) -> Tuple[int, int]:
    """``[first, last)`` global block ids of ``rank``: rank r owns blocks ``[floor(r*B/W), floor((r+1)*B/W))``."""
    assert 0 <= rank < world
    return rank * n_global_blocks // world, (rank + 1) * n_global_blocks // world


def gather_scores(local_scores, n_global_blocks: int, world: int, rank: int, group=None):
    """All ranks' score slices as one tensor in global block order (on the device of ``local_scores``).

    Ranges differ in length by at most one block, so every rank contributes a slice padded to the longest range
    and the padding is dropped after the all-gather."""
    import torch
    import torch.distributed as dist

    lo, hi = rank_block_range(n_global_blocks, world, rank)
    assert local_scores.numel() == hi - lo, "the context must cover exactly this rank's range of blocks"
    if world == 1:
        return local_scores
    longest = max(b - a for a, b in (rank_block_range(n_global_blocks, world, r) for r in range(world)))
    mine = torch.zeros(longest, dtype=local_scores.dtype, device=local_scores.device)
    mine[: hi - lo] = local_scores
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    out = torch.empty(n_global_blocks, dtype=local_scores.dtype, device=local_scores.device)
    for r in range(world):
        a, b = rank_block_range(n_global_blocks, world, r)
        out[a:b] = parts[r][: b - a]
    return out


class ShardedCheckpoint:
    """One rank's part of a running checkpoint that is spread over ``world`` GPUs.

    ``x`` is this rank's slice of the parameters; its blocks (given by ``row_elems`` / ``block_elems`` or
    ``block_offsets``, local offsets) must be exactly the rank's range of the ``n_global_blocks`` global blocks.
    """

    def __init__(self, x, n_global_blocks: int, world: int, rank: int, group=None, n_shards: int = 1,
                 row_elems: int = 0, block_elems: int = 0, block_offsets=None, stream=None):
        self.world, self.rank, self.group = world, rank, group
        self.n_global_blocks = n_global_blocks
        self.first_block, self.last_block = rank_block_range(n_global_blocks, world, rank)
        self.ck = api.ScarCheckpoint(x, n_shards=n_shards, row_elems=row_elems, block_elems=block_elems,
                                     block_offsets=block_offsets, stream=stream)
        if self.ck.n_blocks != self.last_block - self.first_block:
            n = self.ck.n_blocks
            self.ck.close()
            raise ValueError(f"rank {rank} must own {self.last_block - self.first_block} blocks, its layout has {n}")

    def priority_save(self, r: Optional[float] = None, k_global: Optional[int] = None):
        """Checkpoint steps 1 to 4 for the global fraction ``r`` (or ``k_global`` blocks); returns this rank's
        ``scar_save_info`` (``k`` = how many of the selected blocks it owns and has saved)."""
        if k_global is None:
            k_global = api.scar_k_from_r(r, self.n_global_blocks)
        self.ck.block_scores()  # step 1, on the context's stream
        with self._on_stream():
            scores = gather_scores(self.ck.views()["scores"], self.n_global_blocks, self.world, self.rank, self.group)
        self._keep = scores  # alive until the save has read it
        return self.ck.priority_save_sharded(scores, self.n_global_blocks, self.first_block, k_global)

    def _on_stream(self):
        import torch

        return torch.cuda.stream(self.ck._stream)

    def close(self):
        self.ck.close()
