"""ctypes binding of ``libscar.so``: argument marshalling only.

The module-level ``scar_*`` functions mirror ``include/scar.h`` one to one and
take raw device addresses (``int``) or torch CUDA tensors (their ``data_ptr()``
is used).  :class:`ScarCheckpoint` is a small convenience wrapper that owns one
context.  Nothing here computes anything: if the library cannot be loaded the
import of a ``scar_*`` call raises, there is no fallback.
"""

from __future__ import annotations

import ctypes as C
import os
import re
from typing import Optional

import numpy as np

SCAR_F32, SCAR_I32 = 0, 1
SCAR_NORM_DEFAULT, SCAR_NORM_L1 = 0, 1
SCAR_OK = 0

_PKG = os.path.dirname(os.path.abspath(__file__))
_HEADER = os.path.join(os.path.dirname(_PKG), "include", "scar.h")
_lib = None


class ScarError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {scar_strerror(code)} ({code})")
        self.code = code


class scar_layout(C.Structure):
    _fields_ = [("n_elems", C.c_uint64), ("row_elems", C.c_uint64), ("block_elems", C.c_uint32),
                ("n_shards", C.c_uint32), ("block_offsets", C.POINTER(C.c_uint64)), ("n_blocks", C.c_uint64)]


class scar_save_info(C.Structure):
    _fields_ = [("k", C.c_uint64), ("payload_elems", C.c_uint64), ("nonfinite_blocks", C.c_uint64)]


class scar_norm_info(C.Structure):
    _fields_ = [("l2", C.c_double), ("l1", C.c_uint64), ("lost_blocks", C.c_uint64), ("lost_elems", C.c_uint64)]


class scar_drain_view(C.Structure):
    _fields_ = [("info", scar_save_info), ("h_sel", C.c_void_p), ("h_poff", C.c_void_p), ("h_payload", C.c_void_p)]


def lib_path() -> str:
    return os.path.join(_PKG, "libscar.so")


def exported_symbols() -> list:
    """Names of the functions ``include/scar.h`` declares."""
    with open(_HEADER) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(scar_[a-z_0-9]+)\s*\(", text)))


_vp, _u64, _int, _dbl = C.c_void_p, C.c_uint64, C.c_int, C.c_double
_SIGS = {
    "scar_ckpt_init": (_int, [C.POINTER(_vp), _vp, _int, C.POINTER(scar_layout), _vp]),
    "scar_ckpt_init_guarded": (_int, [C.POINTER(_vp), _vp, _int, C.POINTER(scar_layout), _vp]),
    "scar_ckpt_debug_check_guards": (_int, [_vp, C.POINTER(_u64)]),
    "scar_static_debug_check_guard": (_int, [C.POINTER(_u64)]),
    "scar_ckpt_set_norm": (_int, [_vp, _int, _vp]),
    "scar_ckpt_block_scores": (_int, [_vp]),
    "scar_ckpt_priority_save": (_int, [_vp, _dbl, C.POINTER(scar_save_info)]),
    "scar_k_from_r": (_int, [_dbl, _u64, C.POINTER(_u64)]),
    "scar_ckpt_priority_save_k": (_int, [_vp, _u64, C.POINTER(scar_save_info)]),
    "scar_ckpt_priority_save_sharded": (_int, [_vp, _vp, _u64, _u64, _u64, C.POINTER(scar_save_info)]),
    "scar_ckpt_save_round": (_int, [_vp, _u64, C.POINTER(scar_save_info)]),
    "scar_ckpt_save_random": (_int, [_vp, _u64, _vp, C.POINTER(scar_save_info)]),
    "scar_ckpt_round_cursor": (_int, [_vp, C.POINTER(_u64), C.POINTER(_u64)]),
    "scar_recover_partial": (_int, [_vp, _vp, C.POINTER(scar_norm_info)]),
    "scar_recover_partial_blocks": (_int, [_vp, _vp, C.POINTER(scar_norm_info)]),
    "scar_perturbation_norm": (_int, [_vp, _vp, C.POINTER(scar_norm_info)]),
    "scar_perturbation_norm_blocks": (_int, [_vp, _vp, C.POINTER(scar_norm_info)]),
    "scar_perturbation_norm_static": (_int, [_vp, _vp, _int, C.POINTER(scar_layout), _vp, _vp, _vp]),
    "scar_ckpt_priority_save_host": (_int, [_vp, _vp, _dbl, _vp, _vp, _vp, C.POINTER(scar_save_info)]),
    "scar_recover_partial_host": (_int, [_vp, _vp, _vp, C.POINTER(scar_norm_info)]),
    "scar_ckpt_drain_init": (_int, [_vp, _u64, _u64]),
    "scar_ckpt_drain_enqueue": (_int, [_vp, C.POINTER(_u64)]),
    "scar_ckpt_drain_done": (_int, [_vp, _u64]),
    "scar_ckpt_drain_wait": (_int, [_vp, _u64, C.POINTER(scar_drain_view)]),
    "scar_ckpt_drain_release": (_int, [_vp, _u64]),
    "scar_ckpt_store_full": (_int, [_vp, _int]),
    "scar_ckpt_store_drained": (_int, [_vp, _u64, _int]),
    "scar_ckpt_load_stored": (_int, [_vp, _int]),
    "scar_ckpt_load": (_int, [_vp, _vp]),
    "scar_ckpt_last_info": (_int, [_vp, C.POINTER(scar_save_info), C.POINTER(scar_norm_info)]),
    "scar_ckpt_view": (_int, [_vp] + [C.POINTER(_vp)] * 5),
    "scar_ckpt_n_blocks": (_u64, [_vp]),
    "scar_ckpt_launch_count": (_u64, [_vp]),
    "scar_ckpt_profile": (_int, [_vp, _int]),
    "scar_ckpt_profile_read": (_int, [_vp, C.POINTER(C.c_float)]),
    "scar_baseline_iterations": (_dbl, [_dbl, _dbl, _dbl]),
    "scar_discounted_perturbation": (_dbl, [_vp, _vp, _u64, _dbl]),
    "scar_iteration_cost_bound": (_dbl, [_dbl, _dbl, _dbl]),
    "scar_irreducible_error": (_dbl, [_dbl, _dbl]),
    "scar_ckpt_selftest_arm_timeout": (_int, [_vp]),
    "scar_ckpt_debug_select_stamps": (_int, [_vp, C.POINTER(C.c_int64)]),
    "scar_ckpt_destroy": (_int, [_vp]),
    "scar_strerror": (C.c_char_p, [_int]),
}


def load_library():
    """Loads ``libscar.so`` from the package directory; raises if it is not there."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
                               "(there is no CPU fallback)")
        lib = C.CDLL(path)
        for name, (res, args) in _SIGS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _addr(a) -> Optional[int]:
    """Device or host address of ``a``: int, None, torch tensor or numpy array."""
    if a is None:
        return None
    if isinstance(a, int):
        return a
    if isinstance(a, np.ndarray):
        assert a.flags.c_contiguous
        return a.ctypes.data
    if hasattr(a, "data_ptr"):
        assert a.is_contiguous()
        return a.data_ptr()
    raise TypeError(type(a))


def _check(code: int, what: str):
    if code != SCAR_OK:
        raise ScarError(code, what)


def scar_strerror(code: int) -> str:
    return load_library().scar_strerror(code).decode()


def make_layout(n_elems: int, row_elems: int = 0, block_elems: int = 0, n_shards: int = 1,
                block_offsets: Optional[np.ndarray] = None):
    """Builds a ``scar_layout``; keeps the offsets array alive on the returned object."""
    L = scar_layout()
    L.n_elems, L.row_elems, L.block_elems, L.n_shards = n_elems, row_elems, block_elems, n_shards
    if block_offsets is not None:
        off = np.ascontiguousarray(block_offsets, dtype=np.uint64)
        L.block_offsets = off.ctypes.data_as(C.POINTER(C.c_uint64))
        L.n_blocks = off.size - 1
        L._keepalive = off
    return L


def scar_ckpt_init(d_x, dtype: int, layout: scar_layout, cuda_stream: int = 0, guarded: bool = False) -> int:
    ctx = _vp()
    name = "scar_ckpt_init_guarded" if guarded else "scar_ckpt_init"
    _check(getattr(load_library(), name)(C.byref(ctx), _addr(d_x), dtype, C.byref(layout), cuda_stream or None), name)
    return ctx.value


def scar_ckpt_init_guarded(d_x, dtype: int, layout: scar_layout, cuda_stream: int = 0) -> int:
    """``scar_ckpt_init`` for a debug context whose device buffers sit between guard bands."""
    return scar_ckpt_init(d_x, dtype, layout, cuda_stream, guarded=True)


def scar_ckpt_debug_check_guards(ctx: int) -> int:
    """Band bytes of a guarded context that no longer hold the pattern (0 = nothing wrote outside a buffer)."""
    bad = _u64(0)
    _check(load_library().scar_ckpt_debug_check_guards(ctx, C.byref(bad)), "scar_ckpt_debug_check_guards")
    return int(bad.value)


def scar_static_debug_check_guard() -> int:
    bad = _u64(0)
    _check(load_library().scar_static_debug_check_guard(C.byref(bad)), "scar_static_debug_check_guard")
    return int(bad.value)


def scar_ckpt_set_norm(ctx: int, norm: int, h_block_weights: Optional[np.ndarray] = None) -> None:
    w = None if h_block_weights is None else np.ascontiguousarray(h_block_weights, dtype=np.float32)
    _check(load_library().scar_ckpt_set_norm(ctx, norm, _addr(w)), "scar_ckpt_set_norm")


def scar_ckpt_block_scores(ctx: int) -> None:
    _check(load_library().scar_ckpt_block_scores(ctx), "scar_ckpt_block_scores")


def _save_out(sync: bool):
    return scar_save_info() if sync else None


def scar_ckpt_priority_save(ctx: int, r: float, sync: bool = True) -> Optional[scar_save_info]:
    out = _save_out(sync)
    _check(load_library().scar_ckpt_priority_save(ctx, r, C.byref(out) if sync else None), "scar_ckpt_priority_save")
    return out


def scar_k_from_r(r: float, n_blocks: int) -> int:
    """The library's rule for the number of blocks a fraction r stands for."""
    k = _u64(0)
    _check(load_library().scar_k_from_r(r, n_blocks, C.byref(k)), "scar_k_from_r")
    return int(k.value)


def scar_ckpt_priority_save_k(ctx: int, k: int, sync: bool = True) -> Optional[scar_save_info]:
    out = _save_out(sync)
    _check(load_library().scar_ckpt_priority_save_k(ctx, k, C.byref(out) if sync else None),
           "scar_ckpt_priority_save_k")
    return out


def scar_ckpt_priority_save_sharded(ctx: int, d_global_scores, n_global_blocks: int, first_block: int,
                                    k_global: int) -> scar_save_info:
    out = scar_save_info()
    _check(load_library().scar_ckpt_priority_save_sharded(ctx, _addr(d_global_scores), n_global_blocks, first_block,
                                                          k_global, C.byref(out)), "scar_ckpt_priority_save_sharded")
    return out


def scar_ckpt_save_round(ctx: int, k: int, sync: bool = True) -> Optional[scar_save_info]:
    out = _save_out(sync)
    _check(load_library().scar_ckpt_save_round(ctx, k, C.byref(out) if sync else None), "scar_ckpt_save_round")
    return out


def scar_ckpt_save_random(ctx: int, k: int, d_priorities, sync: bool = True) -> Optional[scar_save_info]:
    out = _save_out(sync)
    _check(load_library().scar_ckpt_save_random(ctx, k, _addr(d_priorities), C.byref(out) if sync else None),
           "scar_ckpt_save_random")
    return out


def scar_ckpt_round_cursor(ctx: int, set_to: Optional[int] = None) -> int:
    """Returns the round-robin cursor, after setting it when ``set_to`` is given."""
    got = _u64(0)
    new = _u64(set_to) if set_to is not None else None
    _check(load_library().scar_ckpt_round_cursor(ctx, C.byref(new) if new is not None else None, C.byref(got)),
           "scar_ckpt_round_cursor")
    return int(got.value)


def _norm_call(fn_name: str, ctx: int, mask, sync: bool) -> Optional[scar_norm_info]:
    out = scar_norm_info() if sync else None
    _check(getattr(load_library(), fn_name)(ctx, _addr(mask), C.byref(out) if sync else None), fn_name)
    return out


def scar_recover_partial(ctx: int, h_lost_shards: np.ndarray, sync: bool = True):
    return _norm_call("scar_recover_partial", ctx, np.ascontiguousarray(h_lost_shards, dtype=np.uint8), sync)


def scar_recover_partial_blocks(ctx: int, d_lost_blocks, sync: bool = True):
    return _norm_call("scar_recover_partial_blocks", ctx, d_lost_blocks, sync)


def scar_perturbation_norm(ctx: int, h_lost_shards: Optional[np.ndarray] = None, sync: bool = True):
    m = None if h_lost_shards is None else np.ascontiguousarray(h_lost_shards, dtype=np.uint8)
    return _norm_call("scar_perturbation_norm", ctx, m, sync)


def scar_perturbation_norm_blocks(ctx: int, d_lost_blocks=None, sync: bool = True):
    return _norm_call("scar_perturbation_norm_blocks", ctx, d_lost_blocks, sync)


def scar_perturbation_norm_static(d_x, d_z, dtype: int, layout: scar_layout, d_lost_blocks, d_out,
                                  cuda_stream: int = 0) -> None:
    """Allocation-free perturbation norm: enqueues on ``cuda_stream`` and writes a ``scar_norm_info`` to the
    caller's device buffer ``d_out`` (32 bytes).  See ``include/scar.h`` for who needs it and its limits."""
    _check(load_library().scar_perturbation_norm_static(_addr(d_x), _addr(d_z), dtype, C.byref(layout),
                                                        _addr(d_lost_blocks), _addr(d_out), cuda_stream or None),
           "scar_perturbation_norm_static")


def scar_ckpt_priority_save_host(ctx: int, h_x, r: float, h_payload, h_sel, h_poff) -> scar_save_info:
    out = scar_save_info()
    _check(load_library().scar_ckpt_priority_save_host(ctx, _addr(h_x), r, _addr(h_payload), _addr(h_sel),
                                                       _addr(h_poff), C.byref(out)), "scar_ckpt_priority_save_host")
    return out


def scar_recover_partial_host(ctx: int, h_x, h_lost_shards: np.ndarray) -> scar_norm_info:
    out = scar_norm_info()
    m = np.ascontiguousarray(h_lost_shards, dtype=np.uint8)
    _check(load_library().scar_recover_partial_host(ctx, _addr(h_x), _addr(m), C.byref(out)),
           "scar_recover_partial_host")
    return out


def scar_ckpt_drain_init(ctx: int, max_k: int, max_payload_elems: int) -> None:
    _check(load_library().scar_ckpt_drain_init(ctx, max_k, max_payload_elems), "scar_ckpt_drain_init")


def scar_ckpt_drain_enqueue(ctx: int) -> int:
    t = _u64(0)
    _check(load_library().scar_ckpt_drain_enqueue(ctx, C.byref(t)), "scar_ckpt_drain_enqueue")
    return int(t.value)


def scar_ckpt_drain_done(ctx: int, ticket: int) -> bool:
    rc = load_library().scar_ckpt_drain_done(ctx, ticket)
    if rc < 0:
        raise ScarError(rc, "scar_ckpt_drain_done")
    return bool(rc)


def scar_ckpt_drain_wait(ctx: int, ticket: int, elem_dtype=np.float32) -> dict:
    """Waits for the drain of ``ticket``; returns numpy views (no copy) of the pinned host mirror, valid until
    ``scar_ckpt_drain_release``."""
    v = scar_drain_view()
    _check(load_library().scar_ckpt_drain_wait(ctx, ticket, C.byref(v)), "scar_ckpt_drain_wait")
    k, n = int(v.info.k), int(v.info.payload_elems)

    def view(addr, count, dt):
        if count == 0:
            return np.empty(0, dtype=dt)
        buf = (C.c_char * (count * np.dtype(dt).itemsize)).from_address(addr)
        return np.frombuffer(buf, dtype=dt, count=count)

    return {"info": v.info, "sel": view(v.h_sel, k, np.uint32), "poff": view(v.h_poff, k + 1, np.uint64),
            "payload": view(v.h_payload, n, elem_dtype)}


def scar_ckpt_drain_release(ctx: int, ticket: int) -> None:
    _check(load_library().scar_ckpt_drain_release(ctx, ticket), "scar_ckpt_drain_release")


def scar_ckpt_store_full(ctx: int, fd: int) -> None:
    _check(load_library().scar_ckpt_store_full(ctx, fd), "scar_ckpt_store_full")


def scar_ckpt_store_drained(ctx: int, ticket: int, fd: int) -> None:
    _check(load_library().scar_ckpt_store_drained(ctx, ticket, fd), "scar_ckpt_store_drained")


def scar_ckpt_load_stored(ctx: int, fd: int) -> None:
    _check(load_library().scar_ckpt_load_stored(ctx, fd), "scar_ckpt_load_stored")


def scar_ckpt_load(ctx: int, d_z_src) -> None:
    _check(load_library().scar_ckpt_load(ctx, _addr(d_z_src)), "scar_ckpt_load")


def scar_ckpt_last_info(ctx: int, want_save: bool = True, want_norm: bool = True):
    s = scar_save_info() if want_save else None
    n = scar_norm_info() if want_norm else None
    _check(load_library().scar_ckpt_last_info(ctx, C.byref(s) if s else None, C.byref(n) if n else None),
           "scar_ckpt_last_info")
    return s, n


def scar_ckpt_view(ctx: int) -> dict:
    """Device addresses of z, scores, sel, poff, payload."""
    p = [_vp() for _ in range(5)]
    _check(load_library().scar_ckpt_view(ctx, *[C.byref(q) for q in p]), "scar_ckpt_view")
    return dict(zip(("z", "scores", "sel", "poff", "payload"), (q.value for q in p)))


def scar_ckpt_n_blocks(ctx: int) -> int:
    return int(load_library().scar_ckpt_n_blocks(ctx))


def scar_ckpt_launch_count(ctx: int) -> int:
    return int(load_library().scar_ckpt_launch_count(ctx))


def scar_ckpt_profile(ctx: int, enable: bool) -> None:
    _check(load_library().scar_ckpt_profile(ctx, int(enable)), "scar_ckpt_profile")


def scar_ckpt_profile_read(ctx: int) -> list:
    ms = (C.c_float * 5)()
    _check(load_library().scar_ckpt_profile_read(ctx, ms), "scar_ckpt_profile_read")
    return list(ms)


def scar_baseline_iterations(dist0: float, eps: float, c: float) -> float:
    return float(load_library().scar_baseline_iterations(dist0, eps, c))


def scar_discounted_perturbation(norms, iters, c: float) -> float:
    nrm = np.ascontiguousarray(norms, dtype=np.float64)
    its = np.ascontiguousarray(iters, dtype=np.uint64)
    assert nrm.shape == its.shape and nrm.ndim == 1
    return float(load_library().scar_discounted_perturbation(_addr(nrm) if nrm.size else None,
                                                             _addr(its) if its.size else None, nrm.size, c))


def scar_iteration_cost_bound(delta_T: float, dist0: float, c: float) -> float:
    return float(load_library().scar_iteration_cost_bound(delta_T, dist0, c))


def scar_irreducible_error(delta_max: float, c: float) -> float:
    return float(load_library().scar_irreducible_error(delta_max, c))


def scar_ckpt_selftest_arm_timeout(ctx: int) -> None:
    _check(load_library().scar_ckpt_selftest_arm_timeout(ctx), "scar_ckpt_selftest_arm_timeout")


def scar_ckpt_debug_select_stamps(ctx: int) -> list:
    """Cycle stamps of the last selection kernel (diagnostic builds of the library only)."""
    st = (C.c_int64 * 32)()
    _check(load_library().scar_ckpt_debug_select_stamps(ctx, st), "scar_ckpt_debug_select_stamps")
    return list(st)


def scar_ckpt_destroy(ctx: int) -> None:
    _check(load_library().scar_ckpt_destroy(ctx), "scar_ckpt_destroy")


# ---------------------------------------------------------------------------------------------


class _DevView:
    """Lets torch wrap a raw device address without copying."""

    def __init__(self, addr: int, n: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (addr, False), "version": 3}


def device_array(addr: int, n: int, dtype):
    """A torch tensor aliasing ``n`` elements of ``dtype`` at device address ``addr`` (no copy)."""
    import torch

    np_dt = np.dtype(dtype)
    if n == 0:
        return torch.empty(0, dtype=getattr(torch, np_dt.name), device="cuda")
    return torch.as_tensor(_DevView(addr, n, np_dt.str), device="cuda")


class ScarCheckpoint:
    """One context over a torch CUDA tensor ``x`` (float32 or int32, flat, contiguous)."""

    def __init__(self, x, n_shards: int = 8, row_elems: int = 0, block_elems: int = 0,
                 block_offsets: Optional[np.ndarray] = None, stream=None, guarded: bool = False):
        import torch

        assert x.is_cuda and x.is_contiguous() and x.dim() == 1
        self.dtype = {torch.float32: SCAR_F32, torch.int32: SCAR_I32}[x.dtype]
        self.guarded = guarded
        self.x = x
        self.n_elems = x.numel()
        self._stream = stream if stream is not None else torch.cuda.current_stream(x.device)
        self._layout = make_layout(self.n_elems, row_elems, block_elems, n_shards, block_offsets)
        with torch.cuda.device(x.device):
            self.ctx = scar_ckpt_init(x, self.dtype, self._layout, self._stream.cuda_stream, guarded)
        self.n_blocks = scar_ckpt_n_blocks(self.ctx)

    # views -----------------------------------------------------------------
    def views(self, k: Optional[int] = None, payload_elems: Optional[int] = None) -> dict:
        v = scar_ckpt_view(self.ctx)
        elem = np.float32 if self.dtype == SCAR_F32 else np.int32
        score = np.float32 if self.dtype == SCAR_F32 else np.int64  # bit pattern of uint64 scores
        out = {"z": device_array(v["z"], self.n_elems, elem),
               "scores": device_array(v["scores"], self.n_blocks, score)}
        if k is not None:
            out["sel"] = device_array(v["sel"], k, np.int32)  # bit pattern of uint32 ids
            out["poff"] = device_array(v["poff"], k + 1, np.int64)
            if payload_elems is not None:
                out["payload"] = device_array(v["payload"], payload_elems, elem)
        return out

    # calls -------------------------------------------------------------------
    def set_norm(self, norm: int, block_weights: Optional[np.ndarray] = None):
        if block_weights is not None:
            assert len(block_weights) == self.n_blocks
        scar_ckpt_set_norm(self.ctx, norm, block_weights)

    def check_guards(self) -> int:
        return scar_ckpt_debug_check_guards(self.ctx)

    def block_scores(self):
        scar_ckpt_block_scores(self.ctx)

    def priority_save(self, r: float, sync: bool = True):
        return scar_ckpt_priority_save(self.ctx, r, sync)

    def priority_save_k(self, k: int, sync: bool = True):
        return scar_ckpt_priority_save_k(self.ctx, k, sync)

    def priority_save_sharded(self, d_global_scores, n_global_blocks: int, first_block: int, k_global: int):
        return scar_ckpt_priority_save_sharded(self.ctx, d_global_scores, n_global_blocks, first_block, k_global)

    def save_round(self, k: int, sync: bool = True):
        return scar_ckpt_save_round(self.ctx, k, sync)

    def save_random(self, k: int, d_priorities, sync: bool = True):
        return scar_ckpt_save_random(self.ctx, k, d_priorities, sync)

    def round_cursor(self, set_to: Optional[int] = None) -> int:
        return scar_ckpt_round_cursor(self.ctx, set_to)

    def recover_partial(self, lost_shards: np.ndarray, sync: bool = True):
        return scar_recover_partial(self.ctx, lost_shards, sync)

    def recover_partial_blocks(self, d_lost_blocks, sync: bool = True):
        return scar_recover_partial_blocks(self.ctx, d_lost_blocks, sync)

    def perturbation_norm(self, lost_shards: Optional[np.ndarray] = None, sync: bool = True):
        return scar_perturbation_norm(self.ctx, lost_shards, sync)

    def perturbation_norm_blocks(self, d_lost_blocks=None, sync: bool = True):
        return scar_perturbation_norm_blocks(self.ctx, d_lost_blocks, sync)

    def drain_init(self, max_k: int, max_payload_elems: int):
        scar_ckpt_drain_init(self.ctx, max_k, max_payload_elems)

    def drain_enqueue(self) -> int:
        return scar_ckpt_drain_enqueue(self.ctx)

    def drain_done(self, ticket: int) -> bool:
        return scar_ckpt_drain_done(self.ctx, ticket)

    def drain_wait(self, ticket: int) -> dict:
        return scar_ckpt_drain_wait(self.ctx, ticket, np.float32 if self.dtype == SCAR_F32 else np.int32)

    def drain_release(self, ticket: int):
        scar_ckpt_drain_release(self.ctx, ticket)

    def store_full(self, fd: int):
        scar_ckpt_store_full(self.ctx, fd)

    def store_drained(self, ticket: int, fd: int):
        scar_ckpt_store_drained(self.ctx, ticket, fd)

    def load_stored(self, fd: int):
        scar_ckpt_load_stored(self.ctx, fd)

    def load(self, d_z_src):
        scar_ckpt_load(self.ctx, d_z_src)

    def close(self):
        if getattr(self, "ctx", None):
            scar_ckpt_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
