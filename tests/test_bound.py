"""Iteration-cost arithmetic of Section 3: the oracle against what the paper and brute force fix,
and the library's host-only functions against the oracle (no GPU needed)."""

import math

import numpy as np
import pytest

import oracle


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def iterations_until(x0, c, eps, delta=None, T=None, limit=100000):
    """Brute force on the scalar contraction f(x) = c x (x* = 0): first m with |y^(m)| < eps, where the
    perturbation delta is added to the state just before iteration T is applied (Eq. 2)."""
    y, m = x0, 0
    while not abs(y) < eps:
        if delta is not None and m == T:
            y = y + delta
        y = c * y
        m += 1
        assert m < limit
    return m


@pytest.mark.parametrize("c,x0,eps", [(0.9, 5.0, 1e-6), (0.5, 1.0, 1e-9), (0.99, 100.0, 1e-3)])
def test_baseline_iterations_is_the_linear_rate_count(c, x0, eps):
    # Section 3.1: m > kappa implies |x^(m)| < eps, and for f(x) = c x nothing smaller does
    kappa = oracle.baseline_iterations(x0, eps, c)
    m = iterations_until(x0, c, eps)
    assert m - 1 <= kappa < m + 1e-9
    assert x0 * c ** math.ceil(kappa + 1e-12) <= eps * (1 + 1e-12)


def test_discounted_perturbation_closed_forms():
    assert oracle.discounted_perturbation([], [], 0.9) == 0.0
    assert oracle.discounted_perturbation([3.0], [0], 0.7) == 3.0
    assert oracle.discounted_perturbation([3.0], [2], 0.5) == 12.0  # 3 / 0.25
    assert oracle.discounted_perturbation([1.0, 2.0, 4.0], [0, 1, 2], 0.5) == 1.0 + 4.0 + 16.0
    # constant perturbation at every iteration 0..T: a geometric series
    c, T, d = 0.8, 30, 0.25
    want = d * (c ** -(T + 1) - 1) / (1 / c - 1)
    assert math.isclose(oracle.discounted_perturbation([d] * (T + 1), range(T + 1), c), want, rel_tol=1e-12)


@pytest.mark.parametrize("c,x0,T,delta", [(0.9, 4.0, 50, 0.3), (0.8, 1.0, 10, 2.0), (0.95, 10.0, 120, 1e-2),
                                            (0.5, 3.0, 5, 40.0)])
def test_bound_is_tight_for_a_perturbation_away_from_the_optimum(c, x0, T, delta):
    """Section 3.2 states the bound holds with equality for some deterministic perturbation: on f(x) = c x,
    a push away from the optimum at iteration T delays eps-optimality by exactly the bound (up to the
    rounding of iteration counts to integers)."""
    eps = 1e-7
    base = iterations_until(x0, c, eps)
    pert = iterations_until(x0, c, eps, delta=delta, T=T)
    bound = oracle.iteration_cost_bound(oracle.discounted_perturbation([delta], [T], c), x0, c)
    assert bound > 0
    assert abs((pert - base) - bound) < 1.0 + 1e-9
    # and a push towards the optimum costs less than the bound (the cost may be negative, Section 3)
    toward = iterations_until(x0, c, eps, delta=-min(delta, 0.5 * x0 * c ** T), T=T)
    assert toward - base <= 0 < bound


def test_bound_dominates_random_perturbations_of_a_rotating_contraction():
    """Lemma A.2 / Theorem 3.2 on f(x) = c R x with R orthogonal (so Eq. 5 holds with equality): for random
    perturbations at random iterations the perturbed error never exceeds c^k (||x0|| + Delta_T)."""
    r = rng(3)
    d, c = 6, 0.93
    q, _ = np.linalg.qr(r.standard_normal((d, d)))
    for trial in range(20):
        x0 = r.standard_normal(d)
        when = sorted(r.choice(200, size=5, replace=False).tolist())
        deltas = [r.standard_normal(d) * r.lognormal(-1, 1) for _ in when]
        big = oracle.discounted_perturbation([np.linalg.norm(v) for v in deltas], when, c)
        y = x0.copy()
        for k in range(260):
            if k in when:
                y = y + deltas[when.index(k)]
            y = c * (q @ y)
            if k >= when[-1]:
                assert np.linalg.norm(y) <= c ** (k + 1) * (np.linalg.norm(x0) + big) * (1 + 1e-9)
        eps = 1e-6
        cost_bound = oracle.iteration_cost_bound(big, np.linalg.norm(x0), c)
        kappa = oracle.baseline_iterations(np.linalg.norm(x0), eps, c)
        m = math.floor(kappa + cost_bound) + 1  # any m > kappa + bound must be eps-optimal
        y = x0.copy()
        for k in range(m):
            if k in when:
                y = y + deltas[when.index(k)]
            y = c * (q @ y)
        assert m <= when[-1] or np.linalg.norm(y) < eps * (1 + 1e-9)


def test_bound_limits_and_monotonicity():
    assert oracle.iteration_cost_bound(0.0, 2.0, 0.9) == 0.0
    b = [oracle.iteration_cost_bound(d, 2.0, 0.9) for d in (0.1, 1.0, 10.0, 100.0)]
    assert all(x < y for x, y in zip(b, b[1:]))
    # a worse start makes the same perturbation cheaper; a slower algorithm (c -> 1) pays more iterations
    assert oracle.iteration_cost_bound(1.0, 20.0, 0.9) < oracle.iteration_cost_bound(1.0, 2.0, 0.9)
    assert oracle.iteration_cost_bound(1.0, 2.0, 0.99) > oracle.iteration_cost_bound(1.0, 2.0, 0.9)
    # Delta_T = dist0 costs exactly log 2 / log(1/c) iterations
    assert math.isclose(oracle.iteration_cost_bound(3.0, 3.0, 0.5), 1.0, rel_tol=1e-15)


def test_irreducible_error_is_the_fixed_point_of_constant_perturbations():
    # Example 3.3: pushing by Delta away from the optimum in every iteration of f(x) = c x stalls at c/(1-c) Delta
    c, d = 0.9, 0.01
    y = 5.0
    for _ in range(2000):
        y = c * (y + d)
    assert math.isclose(y, oracle.irreducible_error(d, c), rel_tol=1e-12)
    assert oracle.irreducible_error(0.0, c) == 0.0


# ---- the library's host-only functions against the oracle -------------------------------------


def test_library_bound_functions_match_the_oracle():
    from paper_1810_07354_b200 import api

    r = rng(9)
    for _ in range(200):
        c = float(r.uniform(0.5, 0.999))  # keeps c**-300 well inside the double range
        dist0 = float(r.lognormal(0, 2))
        eps = float(10.0 ** r.uniform(-9, -1))
        n = int(r.integers(0, 6))
        norms = r.lognormal(-2, 2, size=n)
        iters = r.integers(0, 300, size=n)
        d_lib = api.scar_discounted_perturbation(norms, iters, c)
        d_ora = oracle.discounted_perturbation(norms, iters, c)
        assert math.isclose(d_lib, d_ora, rel_tol=1e-12, abs_tol=0.0) or (d_lib == d_ora == 0.0)
        assert math.isclose(api.scar_iteration_cost_bound(d_ora, dist0, c),
                            oracle.iteration_cost_bound(d_ora, dist0, c), rel_tol=1e-12, abs_tol=1e-15)
        assert math.isclose(api.scar_baseline_iterations(dist0, eps, c),
                            oracle.baseline_iterations(dist0, eps, c), rel_tol=1e-12, abs_tol=1e-12)
        assert math.isclose(api.scar_irreducible_error(dist0, c), oracle.irreducible_error(dist0, c), rel_tol=1e-14)


def test_library_bound_functions_reject_bad_arguments():
    from paper_1810_07354_b200 import api

    for c in (0.0, 1.0, -0.5, 1.5, float("nan")):
        assert math.isnan(api.scar_iteration_cost_bound(1.0, 1.0, c))
        assert math.isnan(api.scar_baseline_iterations(1.0, 1e-3, c))
        assert math.isnan(api.scar_discounted_perturbation([1.0], [1], c))
        assert math.isnan(api.scar_irreducible_error(1.0, c))
    assert math.isnan(api.scar_iteration_cost_bound(-1.0, 1.0, 0.5))
    assert math.isnan(api.scar_iteration_cost_bound(1.0, 0.0, 0.5))
    assert math.isnan(api.scar_baseline_iterations(1.0, 0.0, 0.5))
    assert math.isnan(api.scar_discounted_perturbation([-1.0], [0], 0.5))
    assert api.scar_discounted_perturbation([], [], 0.5) == 0.0
