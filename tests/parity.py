"""Comparison protocol between the CUDA library and the CPU oracle (test helper, not collected).

Exactness rules:
  * integer scores / norms, selected ids, payload bytes, offsets, refreshed checkpoint and
    restored buffers are compared bit for bit;
  * float32 block scores and perturbation norms must agree with the fp64 oracle to 1e-5
    relative on the norm (2e-5 on the squared score);
  * selected ids may differ from the oracle's only among blocks whose oracle score lies within
    that tolerance of the k-th largest score; outside the band membership is forced.  When ids
    do differ, what is unique is still checked: the list is the exact top-k (lowest-id ties) of
    the library's own float32 scores, and payload / offsets / checkpoint are exactly x gathered
    over the list.
"""

from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_1810_07354_b200 import api

NORM_RTOL = 1e-5
SQ_RTOL = 2e-5
SQ_ATOL = 1e-30


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def make_ctx(x_dev: torch.Tensor, z_host: np.ndarray, geom=None, boff=None, n_shards=8) -> api.ScarCheckpoint:
    """Context over ``x_dev`` whose running checkpoint is then replaced by ``z_host``.  The context is a guarded
    one: every buffer the library allocates sits between two bands of a known pattern, and ``close`` (see
    conftest.py) fails the test when a kernel has written into a band."""
    if boff is not None:
        ck = api.ScarCheckpoint(x_dev, n_shards=n_shards, block_offsets=boff, guarded=True)
    else:
        ck = api.ScarCheckpoint(x_dev, n_shards=geom.n_shards, row_elems=geom.row_elems, block_elems=geom.block_elems,
                                guarded=True)
    if z_host is not None:
        zt = to_dev(z_host)
        ck.load(zt)
        torch.cuda.synchronize()
    return ck


def same_bits(a: np.ndarray, b: np.ndarray) -> bool:
    """Bytewise equality of two 4-byte-element arrays without building byte strings (NaN-safe)."""
    return a.shape == b.shape and a.dtype.itemsize == b.dtype.itemsize and np.array_equal(
        a.view(np.uint32) if a.dtype.itemsize == 4 else a.view(np.uint64),
        b.view(np.uint32) if b.dtype.itemsize == 4 else b.view(np.uint64))


def check_scores(gpu_scores: np.ndarray, ora_scores: np.ndarray, linear: bool = False):
    """``linear``: the score is itself a norm (l1), so the 1e-5 applies to it directly instead of to its root."""
    if ora_scores.dtype == np.uint64:
        assert gpu_scores.dtype == np.uint64
        np.testing.assert_array_equal(gpu_scores, ora_scores)
        return
    g = gpu_scores.astype(np.float64)
    finite = np.isfinite(ora_scores)
    # non-finite in the oracle must be non-finite on the GPU
    assert not np.any(np.isfinite(g[~finite]))
    o = ora_scores[finite]
    gg = g[finite]
    assert np.all(gg[o == 0.0] == 0.0), "an unchanged block must score exactly 0"
    if linear:
        err, ref = np.abs(gg - o), o
    else:
        err, ref = np.abs(np.sqrt(gg) - np.sqrt(o)), np.sqrt(o)
    bad = err > NORM_RTOL * ref
    assert not bad.any(), f"{bad.sum()} scores off; worst rel {np.max(err[o > 0] / ref[o > 0]):.3e}"


def rank_key(scores: np.ndarray) -> np.ndarray:
    if scores.dtype == np.uint64:
        return scores
    k = scores.astype(np.float64).copy()
    k[~np.isfinite(k)] = np.inf
    return k


def top_k_lowest_id(key: np.ndarray, k: int) -> np.ndarray:
    """Exact top-k with lowest-id ties (numpy, stable sort on the negated rank)."""
    if key.dtype == np.uint64:
        order = np.lexsort((np.arange(key.size), np.uint64(0xFFFFFFFFFFFFFFFF) - key))
    else:
        order = np.lexsort((np.arange(key.size), -key))
    return np.sort(order[:k]).astype(np.uint32)


def check_selection(gpu_sel: np.ndarray, gpu_scores: np.ndarray, ora: "oracle.SaveResult") -> bool:
    """Returns True when the ids equal the oracle's exactly."""
    k, nb = ora.k, ora.scores.size
    assert gpu_sel.dtype == np.uint32 and gpu_sel.size == k
    if k:
        assert int(gpu_sel.max()) < nb
        assert np.all(np.diff(gpu_sel.astype(np.int64)) > 0), "ids must be strictly ascending"
    if np.array_equal(gpu_sel, ora.sel):
        return True
    assert ora.scores.dtype != np.uint64, "integer scores leave no tolerance band"
    key = rank_key(ora.scores)
    tau = np.partition(key, nb - k)[nb - k]
    assert np.isfinite(tau), "non-finite scores tie exactly and leave no freedom"
    hi, lo = tau * (1 + SQ_RTOL) + SQ_ATOL, tau * (1 - SQ_RTOL) - SQ_ATOL
    chosen = np.zeros(nb, dtype=bool)
    chosen[gpu_sel] = True
    assert np.all(chosen[key > hi]), "a block clearly above the threshold was left out"
    assert not np.any(chosen[key < lo]), "a block clearly below the threshold was taken"
    band = (key <= hi) & (key >= lo)
    assert band.sum() > k - int((key > hi).sum()), "the band leaves no freedom, ids must equal the oracle's"
    assert not np.all(key[band] == 0.0), "exact-zero ties are decided by id alone"
    # what is unique: the list is the exact top-k of the library's own scores
    np.testing.assert_array_equal(gpu_sel, top_k_lowest_id(rank_key(gpu_scores), k))
    return False


def fetch_save(ck: api.ScarCheckpoint, info) -> dict:
    v = ck.views(int(info.k), int(info.payload_elems))
    torch.cuda.synchronize()
    out = {name: t.cpu().numpy() for name, t in v.items()}
    out["sel"] = out["sel"].view(np.uint32)
    if out["scores"].dtype == np.int64:
        out["scores"] = out["scores"].view(np.uint64)
    out["poff"] = out["poff"].view(np.uint64)
    return out


def check_save(ck: api.ScarCheckpoint, info, x: np.ndarray, z_before: np.ndarray, boff: np.ndarray,
               ora: "oracle.SaveResult", linear: bool = False) -> dict:
    assert int(info.k) == ora.k
    assert int(info.nonfinite_blocks) == ora.nonfinite_blocks
    got = fetch_save(ck, info)
    check_scores(got["scores"], ora.scores, linear)
    exact = check_selection(got["sel"], got["scores"], ora)
    if exact:
        assert int(info.payload_elems) == ora.payload.size
        np.testing.assert_array_equal(got["poff"], ora.poff)
        assert same_bits(got["payload"], ora.payload), "payload bytes"
        assert same_bits(got["z"], ora.z_after), "refreshed checkpoint"
    else:
        lens = np.diff(boff.astype(np.int64))
        sel = got["sel"].astype(np.int64)
        np.testing.assert_array_equal(got["poff"], np.concatenate([[0], np.cumsum(lens[sel])]).astype(np.uint64))
        ids = np.repeat(np.arange(lens.size), lens)
        chosen = np.zeros(lens.size, dtype=bool)
        chosen[sel] = True
        m = chosen[ids]
        assert same_bits(got["payload"], x[m])
        assert same_bits(got["z"][m], x[m])
        assert same_bits(got["z"][~m], z_before[~m])
    got["exact"] = exact
    return got


def next_checkpoint(z_before: np.ndarray, x: np.ndarray, boff: np.ndarray, got: dict, ora: "oracle.SaveResult"):
    """The running checkpoint the oracle twin continues from after a checked save: the oracle's own when the ids
    were the oracle's, else the oracle's update step applied to the ids the library chose inside the tolerance
    band (already validated).  Never a buffer copied from the device."""
    if got["exact"]:
        return ora.z_after
    z = z_before.copy()
    oracle.update(z, x, boff, np.ascontiguousarray(got["sel"], dtype=np.uint32))
    return z


def check_norm(info, ora: "oracle.NormResult", is_float: bool):
    assert int(info.lost_blocks) == ora.lost_blocks
    assert int(info.lost_elems) == ora.lost_elems
    if is_float:
        assert int(info.l1) == 0
        if np.isfinite(ora.l2):
            assert abs(info.l2 - ora.l2) <= NORM_RTOL * ora.l2, (info.l2, ora.l2)
            if ora.l2 == 0.0:
                assert info.l2 == 0.0
        else:
            assert not np.isfinite(info.l2)
    else:
        assert info.l2 == 0.0 and int(info.l1) == ora.l1
