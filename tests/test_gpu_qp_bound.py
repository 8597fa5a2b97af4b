"""The QP illustration of Section 3.1: per-trial perturbation sizes from the library against fp64, and every
measured iteration cost against the bound of Theorem 3.2."""

import math

import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1810_07354_b200 import qp_bound  # noqa: E402


@pytest.mark.parametrize("mode", ["single", "repeated"])
def test_costs_stay_under_the_bound(mode):
    res = qp_bound.run(trials=300, mode=mode, fail_iter=200, p=0.01, base_iters=400, seed=3, cond=25.0)
    c, dist0 = res["c"], res["dist0"]
    assert math.isclose(c, 0.96, rel_tol=1e-12)
    assert res["baseline_iters"] <= math.floor(res["kappa"]) + 1
    cost, bound, delta_T = res["cost"], res["bound"], res["delta_T"]
    assert np.all(np.isfinite(cost)), "every trial converges once the perturbations stop"
    hit = delta_T > 0
    assert hit.sum() >= (300 if mode == "single" else 200)
    # the library's bound is the oracle's closed form on the same Delta_T
    want = np.array([oracle.iteration_cost_bound(d, dist0, c) for d in delta_T])
    np.testing.assert_allclose(bound, want, rtol=1e-12)
    # Theorem 3.2: past kappa(x, eps) + bound iterations every perturbed run is eps-optimal
    n_pert = cost + res["baseline_iters"]
    assert np.all(n_pert <= np.floor(res["kappa"] + bound) + 1)
    # unperturbed trials cost nothing
    assert np.all(cost[~hit] == 0)
    if mode == "single":
        # a single perturbation at T: Delta_T = c^-T ||delta||, and larger perturbations cost more on average
        order = np.argsort(delta_T)
        assert cost[order[-50:]].mean() > cost[order[:50]].mean()


def test_perturbation_sizes_come_from_block_scores():
    """One round of the harness's measurement by hand: trial t is block t, ||delta_t|| = sqrt(score_t)."""
    from paper_1810_07354_b200 import api

    r = np.random.Generator(np.random.PCG64(5))
    trials = 257
    before = r.standard_normal(trials * 4).astype(np.float32)
    delta = (r.standard_normal(trials * 4) * np.repeat(r.lognormal(0, 1, trials), 4)).astype(np.float32)
    after = (before + delta).astype(np.float32)
    live = torch.from_numpy(after).cuda()
    ck = api.ScarCheckpoint(live, n_shards=1, block_elems=4)
    ck.load(torch.from_numpy(before).cuda())
    ck.block_scores()
    got = np.sqrt(ck.views()["scores"].double().cpu().numpy())
    boff = np.arange(trials + 1, dtype=np.uint64) * 4
    want = np.sqrt(oracle.block_scores(after, before, boff))
    assert np.all(np.abs(got - want) <= 1e-5 * want)
    ck.close()
