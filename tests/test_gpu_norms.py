"""GPU parity of the weighted block norms (Appendix C: length-scaled total variation of topic distributions,
and weighted l2) against the fp64 oracle."""

import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def doc_topic_case(seed, n_docs=6000, topics=100):
    """Document-topic distributions before and after some Gibbs sweeps: document d has L_d tokens (Zipf-like
    lengths); a Binomial(L_d, 0.1) number of its tokens changed topic.  Rows are counts / L_d in float32."""
    r = rng(seed)
    lengths = np.minimum(r.zipf(1.3, n_docs) * 20, 20000).astype(np.int64)
    base = np.stack([r.multinomial(n, r.dirichlet(np.full(topics, 0.2))) for n in lengths])
    now = base.copy()
    for d in range(n_docs):
        for _ in range(r.binomial(lengths[d], 0.1) if d % 3 else 0):  # a third of the documents untouched
            src = r.choice(np.flatnonzero(now[d]))
            now[d, src] -= 1
            now[d, r.integers(0, topics)] += 1
    z = (base / lengths[:, None]).astype(np.float32).ravel()
    x = (now / lengths[:, None]).astype(np.float32).ravel()
    boff = np.arange(n_docs + 1, dtype=np.uint64) * topics
    return x, z, boff, lengths


@pytest.mark.parametrize("topics", [20, 100, 1000])
def test_length_scaled_total_variation_save_and_recovery(topics):
    x, z, boff, lengths = doc_topic_case(50 + topics, n_docs=3000 if topics == 1000 else 6000, topics=topics)
    nb = boff.size - 1
    w = (lengths / 2.0).astype(np.float32)
    xd = parity.to_dev(x)
    ck = api.ScarCheckpoint(xd, n_shards=8, row_elems=topics, block_elems=topics)
    ck.load(parity.to_dev(z))
    ck.set_norm(api.SCAR_NORM_L1, w)
    k = nb // 8
    ora = oracle.save_norm(x, z, boff, k, "l1", w.astype(np.float64))
    info = ck.priority_save_k(k)
    parity.check_save(ck, info, x, z, boff, ora, linear=True)
    # untouched documents score exactly 0 and are never taken while changed ones remain
    assert np.all(ora.scores[::3] == 0.0)
    # recovery legs from the pristine checkpoint
    ck.load(parity.to_dev(z))
    lost = (rng(7).random(nb) < 0.5).astype(np.uint8)
    md = parity.to_dev(lost)
    full = ck.perturbation_norm(None)
    parity.check_norm(full, oracle.perturbation_norm_weighted(x, z, boff, None, "l1", w), True)
    want = oracle.perturbation_norm_weighted(x, z, boff, lost, "l1", w)
    parity.check_norm(ck.perturbation_norm_blocks(md), want, True)
    got = ck.recover_partial_blocks(md)
    parity.check_norm(got, want, True)
    assert got.l2 <= full.l2
    _, x_after = oracle.recover_partial(x, z, boff, lost)
    assert xd.cpu().numpy().tobytes() == x_after.tobytes()
    ck.close()


@pytest.mark.parametrize("norm,name", [(api.SCAR_NORM_DEFAULT, "l2"), (api.SCAR_NORM_L1, "l1")])
def test_weighted_norms_on_ragged_rows(norm, name):
    r = rng(60)
    rows, cols, blk = 40, 5000, 768  # blocks of 768 within rows of 5000: tail of 392, vector path
    n = rows * cols
    z = r.standard_normal(n).astype(np.float32)
    x = (z + r.standard_normal(n).astype(np.float32) * np.repeat(r.lognormal(-3, 1.5, rows), cols).astype(np.float32)).astype(np.float32)
    boff = oracle.layout_offsets(n, cols, blk)
    nb = boff.size - 1
    w = r.uniform(0, 5, nb).astype(np.float32)
    w[::17] = 0.0  # zero weight: such blocks never matter
    xd = parity.to_dev(x)
    ck = api.ScarCheckpoint(xd, n_shards=8, row_elems=cols, block_elems=blk)
    ck.load(parity.to_dev(z))
    ck.set_norm(norm, w)
    for k in (1, nb // 10, nb // 2):
        ck.load(parity.to_dev(z))
        ora = oracle.save_norm(x, z, boff, k, name, w.astype(np.float64))
        info = ck.priority_save_k(k)
        parity.check_save(ck, info, x, z, boff, ora, linear=(name == "l1"))
    ck.load(parity.to_dev(z))
    shards = np.array([0, 1, 0, 0, 1, 0, 0, 1], dtype=np.uint8)
    lost = oracle.expand_shards(nb, shards)
    want = oracle.perturbation_norm_weighted(x, z, boff, lost, name, w)
    parity.check_norm(ck.perturbation_norm(shards), want, True)
    parity.check_norm(ck.recover_partial(shards), want, True)
    # back to the default norm without weights: the plain l2 results
    ck.load(parity.to_dev(z))
    xd.copy_(torch.from_numpy(x))
    ck.set_norm(api.SCAR_NORM_DEFAULT, None)
    parity.check_norm(ck.perturbation_norm(None), oracle.perturbation_norm(x, z, boff, None), True)
    ora = oracle.priority_save(x, z, boff, k=nb // 4)
    parity.check_save(ck, ck.priority_save_k(nb // 4), x, z, boff, ora)
    ck.close()


def test_set_norm_argument_checks():
    xd = torch.zeros(1024, device="cuda")
    ck = api.ScarCheckpoint(xd, n_shards=2, block_elems=64)
    good = np.ones(16, dtype=np.float32)
    ck.set_norm(api.SCAR_NORM_L1, good)
    for bad_value in (-1.0, float("nan"), float("inf")):
        bad = good.copy()
        bad[5] = bad_value
        with pytest.raises(api.ScarError) as e:
            ck.set_norm(api.SCAR_NORM_L1, bad)
        assert e.value.code == -1
    with pytest.raises(api.ScarError):
        api.scar_ckpt_set_norm(ck.ctx, 7, None)
    ck.close()
    xi = torch.zeros(1024, device="cuda", dtype=torch.int32)
    ci = api.ScarCheckpoint(xi, n_shards=2, block_elems=64)
    ci.set_norm(api.SCAR_NORM_L1, None)  # the default for counts already
    with pytest.raises(api.ScarError) as e:
        ci.set_norm(api.SCAR_NORM_L1, good)
    assert e.value.code == -1
    ci.close()
