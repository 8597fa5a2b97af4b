"""CPU oracle for the SCAR checkpoint-and-recover parameter pass (test infrastructure).

Thin ctypes wrapper over ``scar_oracle.c`` plus the step sequencing of one
save / one recovery.  Only tests, the smoke check and the benchmark's CPU
baseline leg may import this package; the CUDA library never does, and this
package never imports the CUDA library or its binding.

All arrays are numpy; element buffers are flat ``float32`` or ``int32``;
``boff`` is the ``uint64[B + 1]`` block-offset array.
"""

from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "scar_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_SO_OMP = os.path.join(_HERE, "liboracle_omp.so")
_lock = threading.Lock()
_lib = None
_lib_omp = None


def build(force: bool = False, openmp: bool = False) -> str:
    """Compile ``scar_oracle.c`` with gcc (strict IEEE: no contraction, no fast-math).

    ``openmp``: the second build of the same file (``-fopenmp``) whose loops over blocks run on all host cores.
    It exists only to be timed as the all-core CPU baseline; pins and parity tests use the plain build."""
    so = _SO_OMP if openmp else _SO
    if force or not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(_SRC):
        tmp = f"{so}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-std=c99", "-Wall", "-Wextra", "-fPIC", "-shared"]
            + (["-fopenmp"] if openmp else []) + ["-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, so)
    return so


_u64, _i64, _dbl, _int = C.c_uint64, C.c_int64, C.c_double, C.c_int
_p = C.c_void_p


_use_openmp = False


def use_openmp(on: bool) -> int:
    """Switches every later call of this package between the plain build and the OpenMP build of the same
    source (for timing the all-core baseline only); returns the number of threads the chosen build uses."""
    global _use_openmp
    _use_openmp = bool(on)
    return int(_load().scar_oracle_threads())


def _load():
    global _lib, _lib_omp
    with _lock:
        if (_lib_omp if _use_openmp else _lib) is None:
            lib = C.CDLL(build(openmp=_use_openmp))
            sig = {
                "scar_oracle_threads": (_int, []),
                "scar_oracle_count_blocks": (_u64, [_u64, _u64, _u64]),
                "scar_oracle_layout_offsets": (None, [_u64, _u64, _u64, _p]),
                "scar_oracle_expand_shards": (None, [_u64, _u64, _p, _p]),
                "scar_oracle_scores_f32": (None, [_p, _p, _p, _u64, _p]),
                "scar_oracle_scores_f32_l1": (None, [_p, _p, _p, _u64, _p]),
                "scar_oracle_scores_i32": (None, [_p, _p, _p, _u64, _p]),
                "scar_oracle_k_from_r": (_i64, [_dbl, _u64]),
                "scar_oracle_select_f64": (_int, [_p, _u64, _u64, _p, _p]),
                "scar_oracle_select_u64": (_int, [_p, _u64, _u64, _p]),
                "scar_oracle_pack": (None, [_p, _p, _p, _u64, _p, _p]),
                "scar_oracle_update": (None, [_p, _p, _p, _p, _u64]),
                "scar_oracle_recover_f32": (_dbl, [_p, _p, _p, _u64, _p, _int, _p, _p]),
                "scar_oracle_recover_i32": (_u64, [_p, _p, _p, _u64, _p, _int, _p, _p]),
            }
            for name, (res, args) in sig.items():
                fn = getattr(lib, name)
                fn.restype, fn.argtypes = res, args
            if _use_openmp:
                _lib_omp = lib
            else:
                _lib = lib
    return _lib_omp if _use_openmp else _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_p)


def _chk(a: np.ndarray, dtype) -> np.ndarray:
    assert a.dtype == np.dtype(dtype) and a.flags.c_contiguous, (a.dtype, dtype)
    return a


def _elem_dtype(x: np.ndarray) -> str:
    if x.dtype == np.float32:
        return "f32"
    if x.dtype == np.int32:
        return "i32"
    raise TypeError(f"element type must be float32 or int32, got {x.dtype}")


# ---- geometry ---------------------------------------------------------------


def layout_offsets(n_elems: int, row_elems: int, block_elems: int) -> np.ndarray:
    lib = _load()
    nb = lib.scar_oracle_count_blocks(n_elems, row_elems, block_elems)
    boff = np.empty(nb + 1, dtype=np.uint64)
    lib.scar_oracle_layout_offsets(n_elems, row_elems, block_elems, _ptr(boff))
    return boff


def expand_shards(n_blocks: int, lost_shards: np.ndarray) -> np.ndarray:
    lost_shards = np.ascontiguousarray(lost_shards, dtype=np.uint8)
    out = np.empty(n_blocks, dtype=np.uint8)
    _load().scar_oracle_expand_shards(n_blocks, lost_shards.size, _ptr(lost_shards), _ptr(out))
    return out


# ---- single steps -------------------------------------------------------------


def ckpt_init(x: np.ndarray) -> np.ndarray:
    """Section 4.2: the running checkpoint starts as a bytewise copy of x^(0)."""
    return x.copy()


def block_scores(x: np.ndarray, z: np.ndarray, boff: np.ndarray) -> np.ndarray:
    """fp64 squared-l2 block scores (float32 data) or uint64 l1 block scores (int32 data)."""
    lib = _load()
    kind = _elem_dtype(x)
    _chk(z, x.dtype), _chk(boff, np.uint64)
    nb = boff.size - 1
    if kind == "f32":
        out = np.empty(nb, dtype=np.float64)
        lib.scar_oracle_scores_f32(_ptr(_chk(x, np.float32)), _ptr(z), _ptr(boff), nb, _ptr(out))
    else:
        out = np.empty(nb, dtype=np.uint64)
        lib.scar_oracle_scores_i32(_ptr(_chk(x, np.int32)), _ptr(z), _ptr(boff), nb, _ptr(out))
    return out


def k_from_r(r: float, n_blocks: int) -> int:
    k = _load().scar_oracle_k_from_r(float(r), n_blocks)
    if k < 0:
        raise ValueError(f"r must lie in [0, 1], got {r}")
    return int(k)


def select_top_k(score: np.ndarray, k: int):
    """Ascending ids of the k highest-scoring blocks (ties to the lowest id); also the non-finite count."""
    lib = _load()
    nb = score.size
    assert 0 <= k <= nb
    sel = np.empty(k, dtype=np.uint32)
    if score.dtype == np.float64:
        bad = _u64(0)
        rc = lib.scar_oracle_select_f64(_ptr(_chk(score, np.float64)), nb, k, _ptr(sel), C.byref(bad))
        nonfinite = int(bad.value)
    else:
        rc = lib.scar_oracle_select_u64(_ptr(_chk(score, np.uint64)), nb, k, _ptr(sel))
        nonfinite = 0
    if rc != 0:
        raise MemoryError("oracle selection could not allocate")
    return sel, nonfinite


def pack(x: np.ndarray, boff: np.ndarray, sel: np.ndarray):
    """Payload (same element type as x) and its ``uint64[k + 1]`` element offsets."""
    lib = _load()
    _elem_dtype(x)
    _chk(sel, np.uint32), _chk(boff, np.uint64)
    lens = (boff[1:] - boff[:-1])[sel.astype(np.int64)]
    total = int(lens.sum())
    payload = np.empty(total, dtype=x.dtype)
    poff = np.empty(sel.size + 1, dtype=np.uint64)
    assert x.flags.c_contiguous
    lib.scar_oracle_pack(_ptr(x), _ptr(boff), _ptr(sel), sel.size, _ptr(payload), _ptr(poff))
    assert int(poff[-1]) == total
    return payload, poff


def update(z: np.ndarray, x: np.ndarray, boff: np.ndarray, sel: np.ndarray) -> None:
    """In place: ``z_b := x_b`` for the selected blocks."""
    _elem_dtype(x)
    _chk(z, x.dtype), _chk(sel, np.uint32), _chk(boff, np.uint64)
    assert z.flags.c_contiguous and x.flags.c_contiguous and z.flags.writeable
    _load().scar_oracle_update(_ptr(z), _ptr(x), _ptr(boff), _ptr(sel), sel.size)


# ---- whole calls ----------------------------------------------------------------


@dataclass
class SaveResult:
    k: int
    scores: np.ndarray  # fp64 or uint64, scores before the save
    sel: np.ndarray  # uint32[k], ascending
    poff: np.ndarray  # uint64[k + 1]
    payload: np.ndarray
    z_after: np.ndarray
    nonfinite_blocks: int


def priority_save(x: np.ndarray, z: np.ndarray, boff: np.ndarray, r: Optional[float] = None,
                  k: Optional[int] = None) -> SaveResult:
    """One prioritized partial checkpoint (Section 4.3, checkpoint steps 1, 3 and 4).

    ``z`` is not modified; the updated running checkpoint is returned.
    """
    nb = boff.size - 1
    if k is None:
        k = k_from_r(r, nb)
    scores = block_scores(x, z, boff)
    sel, bad = select_top_k(scores, k)
    payload, poff = pack(x, boff, sel)
    z_after = z.copy()
    update(z_after, x, boff, sel)
    return SaveResult(k, scores, sel, poff, payload, z_after, bad)


# ---- other norms (Appendix C) -----------------------------------------------------


def block_scores_norm(x: np.ndarray, z: np.ndarray, boff: np.ndarray, norm: str = "l2",
                      weights: Optional[np.ndarray] = None) -> np.ndarray:
    """fp64 block scores of float32 data under a weighted block norm: ``w_b * sum (x - z)^2`` (``"l2"``) or
    ``w_b * sum |x - z|`` (``"l1"``; with ``w_b = L_b / 2`` the length-scaled total variation of Appendix C)."""
    lib = _load()
    _chk(x, np.float32), _chk(z, np.float32), _chk(boff, np.uint64)
    nb = boff.size - 1
    out = np.empty(nb, dtype=np.float64)
    fn = {"l2": lib.scar_oracle_scores_f32, "l1": lib.scar_oracle_scores_f32_l1}[norm]
    fn(_ptr(x), _ptr(z), _ptr(boff), nb, _ptr(out))
    if weights is not None:
        out = out * np.asarray(weights, dtype=np.float64)
    return out


def save_norm(x, z, boff, k: int, norm: str = "l2", weights=None) -> SaveResult:
    """A prioritized save whose distances use the weighted norm above."""
    scores = block_scores_norm(x, z, boff, norm, weights)
    sel, bad = select_top_k(scores, k)
    payload, poff = pack(x, boff, sel)
    z_after = z.copy()
    update(z_after, x, boff, sel)
    return SaveResult(k, scores, sel, poff, payload, z_after, bad)


def perturbation_norm_weighted(x, z, boff, lost_blocks=None, norm: str = "l2", weights=None) -> NormResult:
    """Perturbation of recovering the lost blocks, in the weighted norm: the lost blocks' distances added up
    (the supports are disjoint, proof of Theorem 4.1), square-rooted for l2.  Reported in the ``l2`` field."""
    scores = block_scores_norm(x, z, boff, norm, weights)
    nb = boff.size - 1
    lost = np.ones(nb, dtype=bool) if lost_blocks is None else np.asarray(lost_blocks).astype(bool)
    total = 0.0
    for b in np.flatnonzero(lost):
        total += float(scores[b])
    lens = (boff[1:] - boff[:-1]).astype(np.int64)
    value = float(np.sqrt(total)) if norm == "l2" else total
    return NormResult(value, 0, total, int(lost.sum()), int(lens[lost].sum()))


# ---- baseline selectors of Section 5.4 ---------------------------------------------


def select_round(n_blocks: int, k: int, cursor: int):
    """`round`: the k blocks that follow the cursor, wrapping; returns (ascending ids, next cursor)."""
    assert 0 <= k <= n_blocks and (0 <= cursor < n_blocks or (n_blocks == 0 and cursor == 0))
    ids = [(cursor + j) % n_blocks for j in range(k)]
    nxt = (cursor + k) % n_blocks if n_blocks else 0
    return np.array(sorted(ids), dtype=np.uint32), nxt


def select_random(priorities: np.ndarray, k: int) -> np.ndarray:
    """`random`: the k blocks with the largest caller-drawn uint32 priorities, ties to the lowest id."""
    _chk(priorities, np.uint32)
    sel, _ = select_top_k(priorities.astype(np.uint64), k)
    return sel


def save_selected(x: np.ndarray, z: np.ndarray, boff: np.ndarray, sel: np.ndarray) -> SaveResult:
    """Checkpoint step 4 of Section 4.3 for an id list chosen by any selector; scores are not computed."""
    payload, poff = pack(x, boff, sel)
    z_after = z.copy()
    update(z_after, x, boff, sel)
    return SaveResult(int(sel.size), np.empty(0), sel, poff, payload, z_after, 0)


@dataclass
class NormResult:
    l2: float  # sqrt of the fp64 sum of squares (float data); 0.0 for integer data
    l1: int  # integer l1 sum (integer data); 0 for float data
    sumsq: float
    lost_blocks: int
    lost_elems: int


def _recover(x, z, boff, lost_blocks, write):
    lib = _load()
    kind = _elem_dtype(x)
    _chk(z, x.dtype), _chk(boff, np.uint64)
    assert x.flags.c_contiguous and z.flags.c_contiguous
    nb = boff.size - 1
    if lost_blocks is not None:
        lost_blocks = np.ascontiguousarray(lost_blocks, dtype=np.uint8)
        assert lost_blocks.size == nb
    cb, ce = _u64(0), _u64(0)
    if kind == "f32":
        ss = lib.scar_oracle_recover_f32(_ptr(x), _ptr(z), _ptr(boff), nb, _ptr(lost_blocks), int(write),
                                         C.byref(cb), C.byref(ce))
        return NormResult(float(np.sqrt(ss)), 0, float(ss), int(cb.value), int(ce.value))
    l1 = lib.scar_oracle_recover_i32(_ptr(x), _ptr(z), _ptr(boff), nb, _ptr(lost_blocks), int(write),
                                     C.byref(cb), C.byref(ce))
    return NormResult(0.0, int(l1), 0.0, int(cb.value), int(ce.value))


def perturbation_norm(x, z, boff, lost_blocks=None) -> NormResult:
    """``||z_S - x_S||`` without touching x; ``lost_blocks=None`` is full recovery (Example 2.3)."""
    return _recover(x, z, boff, lost_blocks, write=False)


def recover_partial(x, z, boff, lost_blocks):
    """Partial recovery (Section 4.1): returns the norm and the recovered copy of x."""
    x_after = x.copy()
    res = _recover(x_after, z, boff, lost_blocks, write=True)
    return res, x_after


# ---- iteration-cost arithmetic of Section 3 (plain Python floats, fp64) ---------------


def baseline_iterations(dist0: float, eps: float, c: float) -> float:
    """Section 3.1: iterations after which the unperturbed, linearly convergent sequence is eps-optimal."""
    import math

    return math.log(dist0 / eps) / math.log(1.0 / c)


def discounted_perturbation(norms, iters, c: float) -> float:
    """Theorem 3.2: ``Delta_T = sum_l c**(-l) * E||delta_l||`` over the perturbed iterations."""
    total = 0.0
    for nrm, l in zip(norms, iters):
        total += float(nrm) / (c ** int(l))
    return total


def iteration_cost_bound(delta_T: float, dist0: float, c: float) -> float:
    """Theorem 3.2: ``log(1 + Delta_T / ||x0 - x*||) / log(1 / c)``."""
    import math

    return math.log(1.0 + delta_T / dist0) / math.log(1.0 / c)


def irreducible_error(delta_max: float, c: float) -> float:
    """Example 3.3 (infinite perturbations): accuracy floor ``c / (1 - c) * Delta``."""
    return c / (1.0 - c) * delta_max
