"""scar_perturbation_norm_static: the perturbation norm for callers that cannot allocate.

A recovery handler that runs when device memory is exhausted, or a plug-in whose host framework
forbids cudaMalloc, cannot create a context (scar_ckpt_init allocates the checkpoint copy and its
work arrays).  The static entry point keeps its scratch in a fixed array inside the library, so
these tests check that it gives exactly what the context-based call gives, twice in a row through
the shared scratch, that it refuses layouts beyond its fixed capacity, and that device memory in
use does not grow across a call.  This file sorts last on purpose: a failure here cannot hide the
results of the other GPU tests.
"""

import ctypes as C

import numpy as np
import pytest

import oracle
from workloads import Geometry, block_offsets, make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1810_07354_b200 import api  # noqa: E402


def read_info(d_out: "torch.Tensor") -> api.scar_norm_info:
    raw = d_out.cpu().numpy().tobytes()
    return api.scar_norm_info.from_buffer_copy(raw)


def reference(x, z, geom, mask_dev, dtype_is_float):
    """The existing context-based entry point on the same data."""
    xd = x.clone()
    ck = api.ScarCheckpoint(xd, n_shards=1, row_elems=geom.row_elems, block_elems=geom.block_elems)
    ck.load(z)
    out = ck.perturbation_norm_blocks(mask_dev)
    ck.close()
    return out


@pytest.mark.parametrize("name,kw", [("tiny", dict(n_elems=1 << 20)), ("mf", dict(l_rows=30_000, r_rows=1_000)),
                                      ("lda", dict(vocab=3_000, topics=1000))])
def test_static_norm_matches_context_norm_on_two_calls_in_a_row(name, kw):
    w = make_workload(name, **kw)
    is_float = w.x.dtype == np.float32
    dt = api.SCAR_F32 if is_float else api.SCAR_I32
    x = torch.from_numpy(w.x).cuda()
    z = torch.from_numpy(w.z).cuda()
    nb = w.n_blocks
    rng = np.random.Generator(np.random.PCG64(99))
    masks = [torch.from_numpy((rng.random(nb) < 0.3).astype(np.uint8)).cuda(), None,
             torch.from_numpy((rng.random(nb) < 0.7).astype(np.uint8)).cuda()]
    want = [reference(x, z, w.geom, m, is_float) for m in masks]
    layout = api.make_layout(w.x.size, w.geom.row_elems, w.geom.block_elems, 1)
    d_out = torch.zeros(4, dtype=torch.int64, device="cuda")  # 32 bytes = one scar_norm_info
    stream = torch.cuda.current_stream().cuda_stream
    # first call (does the one-time address look-up), then measure memory around the next ones
    api.scar_perturbation_norm_static(x, z, dt, layout, masks[0], d_out, stream)
    torch.cuda.synchronize()
    got0 = read_info(d_out)
    free_before = torch.cuda.mem_get_info()[0]
    got = [got0]
    for m in masks[1:]:
        api.scar_perturbation_norm_static(x, z, dt, layout, m, d_out, stream)
        torch.cuda.synchronize()
        got.append(read_info(d_out))
    # the figure is device-wide (other processes may free memory meanwhile): it must not have gone down
    assert torch.cuda.mem_get_info()[0] >= free_before, "the call must not take device memory"
    boff = block_offsets(w.geom)
    for g, m in zip(got, masks):  # and against the definition itself, not only against the other entry point
        ora = oracle.perturbation_norm(w.x, w.z, boff, None if m is None else m.cpu().numpy())
        assert (g.lost_blocks, g.lost_elems, g.l1) == (ora.lost_blocks, ora.lost_elems, ora.l1)
        assert abs(g.l2 - ora.l2) <= 1e-5 * ora.l2
    for g, wnt in zip(got, want):
        assert (g.lost_blocks, g.lost_elems, g.l1) == (wnt.lost_blocks, wnt.lost_elems, wnt.l1)
        if is_float:
            assert abs(g.l2 - wnt.l2) <= 1e-5 * wnt.l2
            assert g.l2 == wnt.l2, "same kernels, same order of additions: identical bits expected"
        else:
            assert g.l2 == 0.0
    # inputs are read-only
    assert x.cpu().numpy().tobytes() == w.x.tobytes() and z.cpu().numpy().tobytes() == w.z.tobytes()


@pytest.mark.parametrize("n,row,blk", [
    (1001 * 37, 1001, 256),     # rows of 1001 floats: element-wise path, last block of a row shorter
    (100_000 * 12, 100_000, 1024),  # MLR-shaped rows: 97 full blocks and a tail of 672
    (1 << 20, 0, 1),            # exactly the largest block count the static array holds
])
def test_static_norm_on_other_geometries_twice_in_a_row(n, row, blk):
    """The entry point resolves the geometry and picks its launch shape itself: rows whose last block is
    shorter, blocks that are not 16-byte aligned, and a layout of exactly SCAR_STATIC_MAX_BLOCKS blocks, each
    called twice through the shared array and compared with the context-based call and with the definition."""
    r = np.random.Generator(np.random.PCG64(n + blk))
    geom = Geometry(n, row, blk, 1)
    zh = r.standard_normal(n).astype(np.float32)
    xh = (zh + r.standard_normal(n).astype(np.float32) * np.float32(0.05)).astype(np.float32)
    boff = block_offsets(geom)
    nb = boff.size - 1
    x, z = torch.from_numpy(xh).cuda(), torch.from_numpy(zh).cuda()
    layout = api.make_layout(n, row, blk, 1)
    d_out = torch.zeros(4, dtype=torch.int64, device="cuda")
    for mask_h in ((r.random(nb) < 0.5).astype(np.uint8), None):
        m = None if mask_h is None else torch.from_numpy(mask_h).cuda()
        want = reference(x, z, geom, m, True)
        ora = oracle.perturbation_norm(xh, zh, boff, mask_h)
        for _ in range(2):
            api.scar_perturbation_norm_static(x, z, api.SCAR_F32, layout, m, d_out)
            torch.cuda.synchronize()
            g = read_info(d_out)
            assert (g.lost_blocks, g.lost_elems) == (want.lost_blocks, want.lost_elems) == (ora.lost_blocks, ora.lost_elems)
            assert g.l2 == want.l2 and abs(g.l2 - ora.l2) <= 1e-5 * ora.l2


def test_a_warmed_up_static_call_changes_nothing_it_should_not():
    """A zero-size call is a complete warm-up (it looks the array's address up and loads the module that holds
    it); after it, a real call leaves device memory in use as it was."""
    d_out = torch.ones(4, dtype=torch.int64, device="cuda")
    empty = api.make_layout(0, 0, 256, 1)
    api.scar_perturbation_norm_static(None, None, api.SCAR_F32, empty, None, d_out)
    torch.cuda.synchronize()
    assert d_out.cpu().tolist() == [0, 0, 0, 0]
    buf = torch.arange(1 << 14, dtype=torch.float32, device="cuda")
    zero = torch.zeros(1 << 14, dtype=torch.float32, device="cuda")
    before = torch.cuda.mem_get_info()[0]
    api.scar_perturbation_norm_static(buf, zero, api.SCAR_F32, api.make_layout(1 << 14, 0, 128, 1), None, d_out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= before
    info = read_info(d_out)
    want = float(np.sqrt(np.sum(np.arange(1 << 14, dtype=np.float64) ** 2)))
    assert abs(info.l2 - want) <= 1e-5 * want and info.lost_blocks == 128


def test_static_norm_rejects_what_it_cannot_hold():
    lib = api.load_library()
    d_out = torch.zeros(4, dtype=torch.int64, device="cuda")
    buf = torch.zeros(1 << 12, dtype=torch.float32, device="cuda")
    too_many = api.make_layout((1 << 20) + 1, 0, 1, 1)  # one block more than SCAR_STATIC_MAX_BLOCKS
    rc = lib.scar_perturbation_norm_static(buf.data_ptr(), buf.data_ptr(), 0, C.byref(too_many), None,
                                           d_out.data_ptr(), None)
    assert rc == -7 and "fixed-size" in api.scar_strerror(rc)
    explicit = api.make_layout(8, block_offsets=np.array([0, 4, 8], dtype=np.uint64))
    assert lib.scar_perturbation_norm_static(buf.data_ptr(), buf.data_ptr(), 0, C.byref(explicit), None,
                                             d_out.data_ptr(), None) == -1
    ok = api.make_layout(1 << 12, 0, 256, 1)
    assert lib.scar_perturbation_norm_static(buf.data_ptr() + 4, buf.data_ptr(), 0, C.byref(ok), None,
                                             d_out.data_ptr(), None) == -1, "misaligned x"
    assert lib.scar_perturbation_norm_static(buf.data_ptr(), buf.data_ptr(), 0, C.byref(ok), None, None, None) == -1
    # a valid call right after the refusals still works: x == z gives a zero perturbation
    api.scar_perturbation_norm_static(buf, buf, api.SCAR_F32, ok, None, d_out)
    torch.cuda.synchronize()
    info = read_info(d_out)
    assert info.l2 == 0.0 and info.lost_blocks == 16 and info.lost_elems == 1 << 12


def test_nothing_was_written_behind_the_static_array():
    """Runs after the calls above: the band behind the library's fixed array still holds its pattern."""
    assert api.scar_static_debug_check_guard() == 0
