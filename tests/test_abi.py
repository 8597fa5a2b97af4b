"""CPU-side checks of the C ABI: the library builds, loads and exports what the header declares.

No compute call is made here; only argument validation that happens before any CUDA work.
"""

import ctypes as C
import os

import pytest

from paper_1810_07354_b200 import _build, api


@pytest.fixture(scope="module")
def lib():
    _build.build()
    return api.load_library()


def test_header_declares_the_four_named_calls():
    names = api.exported_symbols()
    for n in ("scar_ckpt_init", "scar_ckpt_priority_save", "scar_recover_partial", "scar_perturbation_norm"):
        assert n in names


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = api.exported_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in scar.h but not exported by libscar.so"
        assert n in api._SIGS, f"{n} has no ctypes signature"
        assert hasattr(api, n), f"{n} has no Python binding of the same name"
    assert set(api._SIGS) == set(names), "binding and header disagree"


def test_library_is_in_tree():
    assert os.path.dirname(api.lib_path()) == os.path.dirname(os.path.abspath(api.__file__))


def test_strerror(lib):
    assert api.scar_strerror(0) == "ok"
    seen = {api.scar_strerror(c) for c in range(-6, 1)}
    assert len(seen) == 7
    assert api.scar_strerror(-99) == "unknown error"


def test_init_rejects_bad_arguments_before_touching_cuda(lib):
    ctx = C.c_void_p(123)
    L = api.make_layout(1024, 0, 256, 8)
    assert lib.scar_ckpt_init(None, None, 0, C.byref(L), None) == -1
    assert lib.scar_ckpt_init(C.byref(ctx), None, 0, None, None) == -1 and ctx.value is None
    assert lib.scar_ckpt_init(C.byref(ctx), None, 0, C.byref(L), None) == -1, "NULL x with elements"
    assert lib.scar_ckpt_init(C.byref(ctx), 0x1004, 0, C.byref(L), None) == -1, "x must be 16-byte aligned"
    assert lib.scar_ckpt_init(C.byref(ctx), 0x1000, 7, C.byref(L), None) == -1, "unknown dtype"


@pytest.mark.parametrize("kw", [
    dict(n_elems=1024, row_elems=0, block_elems=0, n_shards=8),     # zero block length
    dict(n_elems=1024, row_elems=100, block_elems=10, n_shards=8),  # rows do not tile the buffer
    dict(n_elems=1024, row_elems=2048, block_elems=10, n_shards=8),  # row longer than the buffer
    dict(n_elems=1024, row_elems=0, block_elems=256, n_shards=0),   # no shards
    dict(n_elems=1 << 40, row_elems=0, block_elems=1, n_shards=1),  # more than 2^32 - 1 blocks
])
def test_init_rejects_bad_layouts(lib, kw):
    ctx = C.c_void_p()
    L = api.make_layout(**kw)
    assert lib.scar_ckpt_init(C.byref(ctx), 0x1000, 0, C.byref(L), None) == -2


@pytest.mark.parametrize("off", [[1, 4, 8], [0, 5, 4, 8], [0, 4, 9]])
def test_init_rejects_bad_explicit_offsets(lib, off):
    import numpy as np

    ctx = C.c_void_p()
    L = api.make_layout(8, block_offsets=np.array(off, dtype=np.uint64))
    assert lib.scar_ckpt_init(C.byref(ctx), 0x1000, 0, C.byref(L), None) == -2


def test_null_context_is_an_error_everywhere(lib):
    assert lib.scar_ckpt_block_scores(None) == -1
    assert lib.scar_ckpt_priority_save(None, 0.5, None) == -1
    assert lib.scar_ckpt_priority_save_k(None, 1, None) == -1
    assert lib.scar_recover_partial(None, None, None) == -1
    assert lib.scar_perturbation_norm(None, None, None) == -1
    assert lib.scar_ckpt_destroy(None) == -1
    assert lib.scar_ckpt_n_blocks(None) == 0 and lib.scar_ckpt_launch_count(None) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "lib_path", lambda: str(tmp_path / "libscar.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        api.scar_ckpt_n_blocks(0)
