"""Running-checkpoint simulator: the experiments of Sections 5.3 and 5.4 on a synthetic
iterative-convergent algorithm.

A parameter vector ``x`` lives in device memory and is advanced by a caller-supplied update ``f``
(Eq. 1).  Every ``period`` iterations a partial checkpoint of ``k`` blocks is taken with one of the
three selectors the paper compares (``priority``, ``round``, ``random``; Section 5.4), keeping the
data written per ``C`` iterations constant: ``k = round(r B)`` blocks every ``r C`` iterations
(Section 4.2).  At a failure iteration a set of blocks is lost and restored from the running
checkpoint (partial recovery, Section 4.1); the perturbation norm the library reports feeds the bound
of Theorem 3.2, and the run continues until it is ``eps``-optimal to measure the rework iterations.

All checkpoint and recovery work runs in the library (``api.ScarCheckpoint``); torch is used for the
training update itself, which is the caller's code, and for random draws.

    python -m paper_1810_07354_b200.simulate --n-blocks 65536 --block 256 --trials 20
"""

from __future__ import annotations

import argparse
import json
import math
from dataclasses import dataclass, field
from typing import Callable, Optional

import numpy as np

from . import api

STRATEGIES = ("priority", "round", "random")


@dataclass
class SeparableQuadratic:
    """Gradient descent with step 1/L on ``l(x) = 1/2 sum_i a_i (x_i - x*_i)^2``: the update is
    ``x <- x* + rate * (x - x*)`` with ``rate_i = 1 - a_i / L`` in ``[0, c]``, so the iterates converge
    linearly with ``c = max rate`` (Eq. 5) and strong convexity gives Eq. 6 (Lemma 3.1)."""

    x_star: "object"  # torch tensors on the device
    rate: "object"

    @property
    def c(self) -> float:
        return float(self.rate.max())

    def step(self, x) -> None:
        x.sub_(self.x_star).mul_(self.rate).add_(self.x_star)

    def error(self, x) -> float:
        import torch

        return float(torch.linalg.vector_norm((x - self.x_star).double()))


def make_quadratic(n_blocks: int, block: int, seed: int, c_lo: float = 0.80, c_hi: float = 0.995, device="cuda"):
    """Per-block contraction rates spread log-uniformly in ``1 - rate`` over ``[1 - c_hi, 1 - c_lo]``: some
    blocks settle within tens of iterations, others keep moving for a thousand, which is what makes the choice of
    blocks to checkpoint matter.  Returns ``(problem, x0)``."""
    import torch

    g = torch.Generator(device=device).manual_seed(seed)
    n = n_blocks * block
    u = torch.rand(n_blocks, device=device, generator=g)
    gap = torch.exp(math.log(1 - c_hi) + u * (math.log(1 - c_lo) - math.log(1 - c_hi)))
    rate = (1 - gap).float().repeat_interleave(block).contiguous()
    x_star = torch.randn(n, device=device, generator=g)
    x0 = x_star + torch.randn(n, device=device, generator=g)
    return SeparableQuadratic(x_star, rate), x0.contiguous()


@dataclass
class Simulation:
    """One training run with a running checkpoint.  ``iterate()`` applies one update and, when the
    schedule says so, one partial checkpoint; ``fail()`` loses a set of blocks and recovers them."""

    x: "object"
    step: Callable
    block: int
    strategy: str = "priority"
    r: float = 1.0
    full_period: int = 8  # C: iterations between FULL checkpoints at r = 1
    seed: int = 0
    iteration: int = 0
    saves: int = 0
    saved_blocks: int = 0
    ck: Optional[api.ScarCheckpoint] = None
    _gen: "object" = field(default=None, repr=False)

    def __post_init__(self):
        import torch

        assert self.strategy in STRATEGIES and 0.0 < self.r <= 1.0
        self.ck = api.ScarCheckpoint(self.x, n_shards=1, block_elems=self.block)  # z := x^(0), Section 4.2
        self.n_blocks = self.ck.n_blocks
        # blocks per save and iterations between saves: both by the library's own rounding rule for a fraction
        self.k = api.scar_k_from_r(self.r, self.n_blocks)
        self.period = api.scar_k_from_r(self.r, self.full_period)
        self._gen = torch.Generator(device=self.x.device).manual_seed(self.seed)

    def draw_priorities(self):
        """The random selector's draw: one uniform 31-bit priority per block from the seeded device generator."""
        import torch

        return torch.randint(0, 2**31 - 1, (self.n_blocks,), device=self.x.device, generator=self._gen,
                             dtype=torch.int32)

    def checkpoint_due_next(self) -> bool:
        return (self.iteration + 1) % self.period == 0

    def iterate(self, priorities=None):
        """One update of the training algorithm; returns the save info when a checkpoint followed it.
        ``priorities`` (random selector only) replaces the simulator's own draw for that checkpoint."""
        self.step(self.x)
        self.iteration += 1
        if self.iteration % self.period:
            return None
        return self.checkpoint(priorities)

    def checkpoint(self, priorities=None):
        if self.strategy == "priority":
            info = self.ck.priority_save_k(self.k)
        elif self.strategy == "round":
            info = self.ck.save_round(self.k)
        else:
            info = self.ck.save_random(self.k, priorities if priorities is not None else self.draw_priorities())
        self.saves += 1
        self.saved_blocks += int(info.k)
        return info

    def fail(self, d_lost_blocks, partial: bool = True):
        """Loses the masked blocks at the current iteration.  Partial recovery restores only those; the
        traditional scheme (``partial=False``) rolls every block back.  Returns ``(norm_of_recovery, full_norm)``:
        the perturbation actually incurred and the one a full recovery would have incurred (Theorem 4.1)."""
        full = self.ck.perturbation_norm(None)
        if partial:
            got = self.ck.recover_partial_blocks(d_lost_blocks)
        else:
            got = self.ck.recover_partial(np.ones(1, dtype=np.uint8))
        return got, full

    def close(self):
        if self.ck is not None:
            self.ck.close()
            self.ck = None


def run_trial(problem: SeparableQuadratic, x0, block: int, strategy: str, r: float, full_period: int,
              fail_iter: int, lost_frac: float, eps: float, seed: int, partial: bool = True,
              baseline_iters: Optional[int] = None, max_iters: int = 20000) -> dict:
    """One failure experiment (Sections 5.3 / 5.4): returns the perturbation norms, the bound of Theorem 3.2
    and the measured rework iterations against the unperturbed run.

    ``eps`` must stay above the float32 floor of the update: an element stops moving once
    ``(1 - rate) |x - x*|`` drops below half an ulp of ``x*`` (the reduced-precision perturbation of Example 2.1),
    so a run asked for more accuracy than that never becomes eps-optimal and stops at ``max_iters``
    (``converged`` is then false)."""
    import torch

    x = x0.clone()
    sim = Simulation(x, problem.step, block, strategy, r, full_period, seed)
    g = torch.Generator(device=x.device).manual_seed(seed + 7919)
    dist0 = problem.error(x)
    while sim.iteration < fail_iter:
        sim.iterate()
    lost = (torch.rand(sim.n_blocks, device=x.device, generator=g) < lost_frac).to(torch.uint8)
    got, full = sim.fail(lost, partial)
    while problem.error(x) >= eps and sim.iteration < max_iters:
        sim.iterate()
    c = problem.c
    converged = problem.error(x) < eps
    n_base = baseline_iters if baseline_iters is not None else unperturbed_iterations(problem, x0, eps, max_iters)
    delta_T = api.scar_discounted_perturbation([got.l2], [fail_iter], c)
    out = {"strategy": strategy, "r": r, "k": sim.k, "period": sim.period, "fail_iter": fail_iter,
           "lost_blocks": int(got.lost_blocks), "perturbation": got.l2, "full_perturbation": full.l2,
           "rework_iters": sim.iteration - n_base, "baseline_iters": n_base,
           "bound_iters": api.scar_iteration_cost_bound(delta_T, dist0, c), "c": c, "dist0": dist0, "eps": eps,
           "converged": bool(converged), "saves": sim.saves,
           "saved_blocks": sim.saved_blocks}
    sim.close()
    return out


def unperturbed_iterations(problem: SeparableQuadratic, x0, eps: float, max_iters: int = 20000) -> int:
    """Iterations the update needs from ``x0`` to come within ``eps`` with no failure, counted exactly."""
    base = x0.clone()
    n = 0
    while problem.error(base) >= eps and n < max_iters:
        problem.step(base)
        n += 1
    return n


def main(argv=None):
    import torch

    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--n-blocks", type=int, default=4096)
    ap.add_argument("--block", type=int, default=256)
    ap.add_argument("--trials", type=int, default=10)
    ap.add_argument("--full-period", type=int, default=64, help="C: iterations between full checkpoints")
    ap.add_argument("--fractions", type=float, nargs="+", default=[1.0, 0.5, 0.25, 0.125])
    ap.add_argument("--lost-frac", type=float, default=0.5)
    ap.add_argument("--fail-p", type=float, default=0.01, help="parameter of the geometric failure time")
    ap.add_argument("--eps-rel", type=float, default=1e-4,
                    help="eps as a fraction of ||x0 - x*|| (keep it above the float32 floor of the update)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--json", action="store_true", help="print one JSON line per trial instead of the summary")
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: there is no CPU path")
    problem, x0 = make_quadratic(a.n_blocks, a.block, a.seed)
    fail_iters = np.random.Generator(np.random.PCG64(a.seed)).geometric(a.fail_p, size=a.trials)
    eps = a.eps_rel * problem.error(x0)
    n_base = unperturbed_iterations(problem, x0, eps)
    rows = []
    for strategy in STRATEGIES:
        for r in a.fractions:
            for t in range(a.trials):
                res = run_trial(problem, x0, a.block, strategy, r, a.full_period, int(fail_iters[t]), a.lost_frac,
                                eps, a.seed + t, baseline_iters=n_base)
                if a.json:
                    print(json.dumps(res))
                rows.append(res)
    # traditional scheme: full checkpoints, full recovery
    for t in range(a.trials):
        res = run_trial(problem, x0, a.block, "priority", 1.0, a.full_period, int(fail_iters[t]), a.lost_frac,
                        eps, a.seed + t, partial=False, baseline_iters=n_base)
        res["strategy"] = "full-recovery"
        if a.json:
            print(json.dumps(res))
        rows.append(res)
    if not a.json:
        print(f"{a.n_blocks} blocks of {a.block}, c = {problem.c:.4f}, eps = {eps:.3g}, unperturbed run: {n_base} iterations, "
              f"{a.trials} trials, failure time ~ Geometric({a.fail_p}), {a.lost_frac:.0%} of the blocks lost")
        print(f"{'strategy':>14} {'r':>6} {'period':>6} {'rework iters':>13} {'bound':>8} {'|delta|':>10} {'|delta| full':>12}")
        seen = []
        for res in rows:
            key = (res["strategy"], res["r"])
            if key in seen:
                continue
            seen.append(key)
            grp = [q for q in rows if (q["strategy"], q["r"]) == key]
            m = lambda f: float(np.mean([q[f] for q in grp]))  # noqa: E731
            print(f"{key[0]:>14} {key[1]:>6.3f} {grp[0]['period']:>6d} {m('rework_iters'):>13.1f} "
                  f"{m('bound_iters'):>8.1f} {m('perturbation'):>10.4g} {m('full_perturbation'):>12.4g}")
    return rows


if __name__ == "__main__":
    main()
