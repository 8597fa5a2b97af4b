"""The running-checkpoint simulator in lock-step with a twin built from the CPU oracle: same updates, same
checkpoints, same failure, compared after every library call."""

import math

import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import parity  # noqa: E402
from paper_1810_07354_b200 import api, simulate  # noqa: E402


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


@pytest.mark.parametrize("strategy", simulate.STRATEGIES)
def test_simulation_in_lockstep_with_the_oracle(strategy):
    nb, blk = 768, 96
    problem, x0 = simulate.make_quadratic(nb, blk, seed=3)
    x = x0.clone()
    sim = simulate.Simulation(x, problem.step, blk, strategy, r=0.25, full_period=12, seed=5)
    assert sim.k == 192 and sim.period == 3
    xs, rate = problem.x_star.cpu().numpy(), problem.rate.cpu().numpy()
    hx = x0.cpu().numpy().copy()
    hz = oracle.ckpt_init(hx)
    boff = (np.arange(nb + 1, dtype=np.uint64) * blk)
    cursor, r = 0, rng(17)
    for it in range(1, 46):
        pri = sim.draw_priorities() if strategy == "random" and sim.checkpoint_due_next() else None
        info = sim.iterate(pri)
        hx = ((hx - xs) * rate + xs).astype(np.float32)  # the same three float32 roundings as the device update
        assert x.cpu().numpy().tobytes() == hx.tobytes(), f"parameters diverged at iteration {it}"
        assert (info is not None) == (it % 3 == 0)
        if info is not None:
            if strategy == "priority":
                ora = oracle.priority_save(hx, hz, boff, k=sim.k)
                got = parity.check_save(sim.ck, info, hx, hz, boff, ora)
                hz = parity.next_checkpoint(hz, hx, boff, got, ora)  # the validated ids decide what it holds
            else:
                if strategy == "round":
                    sel, cursor = oracle.select_round(nb, sim.k, cursor)
                else:
                    sel = oracle.select_random(pri.cpu().numpy().view(np.uint32), sim.k)
                ora = oracle.save_selected(hx, hz, boff, sel)
                got = parity.fetch_save(sim.ck, info)
                np.testing.assert_array_equal(got["sel"], ora.sel)
                np.testing.assert_array_equal(got["poff"], ora.poff)
                assert parity.same_bits(got["payload"], ora.payload) and parity.same_bits(got["z"], ora.z_after)
                hz = ora.z_after
        if it == 28:  # failure between two checkpoints: half of the blocks are lost
            lost = (r.random(nb) < 0.5).astype(np.uint8)
            want_full = oracle.perturbation_norm(hx, hz, boff, None)
            want, hx = oracle.recover_partial(hx, hz, boff, lost)
            got_n, full_n = sim.fail(parity.to_dev(lost))
            parity.check_norm(full_n, want_full, True)
            parity.check_norm(got_n, want, True)
            assert got_n.l2 <= full_n.l2  # Theorem 4.1
            assert x.cpu().numpy().tobytes() == hx.tobytes()
    assert sim.saves == 15 and sim.saved_blocks == 15 * 192
    sim.close()


def test_trial_report_is_consistent_with_theorem_3_2():
    problem, x0 = simulate.make_quadratic(256, 64, seed=1, c_lo=0.6, c_hi=0.95)
    for strategy in simulate.STRATEGIES:
        res = simulate.run_trial(problem, x0, 64, strategy, r=0.25, full_period=16, fail_iter=40, lost_frac=0.5,
                                 eps=1e-4, seed=2)
        c = res["c"]
        assert 0.9 < c < 0.95 and res["k"] == 64 and res["period"] == 4
        assert 0.0 < res["perturbation"] <= res["full_perturbation"]  # Theorem 4.1
        delta_T = oracle.discounted_perturbation([res["perturbation"]], [40], c)
        want = oracle.iteration_cost_bound(delta_T, res["dist0"], c)
        assert math.isclose(res["bound_iters"], want, rel_tol=1e-9)
        # Theorem 3.2: past kappa(x, eps) + bound iterations the perturbed run is eps-optimal
        kappa = oracle.baseline_iterations(res["dist0"], res["eps"], c)
        assert res["baseline_iters"] <= math.floor(kappa) + 1
        assert res["baseline_iters"] + res["rework_iters"] <= math.floor(kappa + want) + 1
        assert res["rework_iters"] >= 0  # a reset towards older values does not speed this problem up
    full = simulate.run_trial(problem, x0, 64, "priority", r=1.0, full_period=16, fail_iter=40, lost_frac=0.5,
                              eps=1e-4, seed=2, partial=False)
    assert full["lost_blocks"] == 256 and math.isclose(full["perturbation"], full["full_perturbation"], rel_tol=1e-12)
