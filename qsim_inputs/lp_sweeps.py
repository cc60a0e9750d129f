"""Grids of steady-state LPs for the planning studies of the paper's Section 6.3 ("The Cost of Service Quality and
Hardware Resources"): Pareto frontiers of revenue against one service-level indicator at a time (prefill fairness eta_1,
Eq. (39); decode fairness eta_2, Eq. (41); average time per output token eta_3, Eq. (43)), and the sensitivity of revenue
and average TPOT to the decode cap B and to the iteration-time parameters alpha, beta (tau_mix = alpha + beta C) and
gamma = 1 / tau_solo.  Host-side set-up work (every grid point is one small LP); the simulators are not involved.

The instance is the paper's two-class synthetic one (EC, "Convergence Analysis"): P = (300, 3000), D = (1000, 400),
lambda = (0.5, 0.5), theta = (0.1, 0.1), separate charging with c_p = 0.1, c_d = 0.2, C = 256, alpha = 0.0174,
beta = 6.2e-5; B = 16 and tau_solo = 0.022 s as elsewhere in this repository (the paper states neither for this study).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

from . import fluid_lp as lp


@dataclass(frozen=True)
class Instance:
    P: tuple = (300.0, 3000.0)
    D: tuple = (1000.0, 400.0)
    lam: tuple = (0.5, 0.5)
    theta: tuple = (0.1, 0.1)
    c_p: float = 0.1
    c_d: float = 0.2
    separate: bool = True
    B: int = 16
    C: int = 256
    alpha: float = 0.0174
    beta: float = 6.2e-5
    gamma: float = 1.0 / 0.022

    @property
    def tau_mix(self) -> float:
        return self.alpha + self.beta * self.C

    @property
    def tau_solo(self) -> float:
        return 1.0 / self.gamma


def average_tpot(inst: Instance, x_total: float) -> float:
    """Left side of Eq. (43): decode-slot-weighted mean iteration time when a fraction x_total of the GPUs is mixed."""
    B = inst.B
    num = inst.tau_mix * (B - 1) * x_total + inst.tau_solo * B * (1.0 - x_total)
    den = (B - 1) * x_total + B * (1.0 - x_total)
    return num / den


def solve(inst: Instance, **sli):
    """One LP; returns (revenue per GPU, plan) or (nan, None) when the constraint set is empty."""
    try:
        plan = lp.solve_plan(inst.lam, inst.P, inst.D, inst.theta, inst.B, inst.C, inst.tau_mix, inst.tau_solo,
                             inst.c_p, inst.c_d, separate=inst.separate, **sli)
    except RuntimeError:
        return float("nan"), None
    return plan.value, plan


def frontier(inst: Instance, indicator: str, etas) -> np.ndarray:
    """Revenue per GPU along one indicator: 'prefill_fair' (eta_1), 'decode_fair' (eta_2) or 'tpot_cap' (eta_3), each
    with q_d = 0 as the SLI-aware planning problem requires (Section 5.2); nan where no plan satisfies the target."""
    assert indicator in ("prefill_fair", "decode_fair", "tpot_cap")
    return np.array([solve(inst, qd_zero=True, **{indicator: float(e)})[0] for e in etas])


def shadow_price(etas, revenue) -> np.ndarray:
    """Slope of a frontier: revenue given up per unit of a stricter target (finite differences between grid points)."""
    etas = np.asarray(etas, float)
    revenue = np.asarray(revenue, float)
    return np.diff(revenue) / np.diff(etas)


def sensitivity(inst: Instance, parameter: str, values):
    """Revenue per GPU and average TPOT of the unconstrained plan as one of B, alpha, beta, gamma varies."""
    assert parameter in ("B", "alpha", "beta", "gamma")
    rev, tpot = [], []
    for v in values:
        cur = replace(inst, **{parameter: int(v) if parameter == "B" else float(v)})
        r, plan = solve(cur)
        rev.append(r)
        tpot.append(average_tpot(cur, float(plan.x.sum())) if plan is not None else float("nan"))
    return np.array(rev), np.array(tpot)


def grid(inst: Instance, p1: str, v1, p2: str, v2) -> np.ndarray:
    """Revenue per GPU over a two-parameter grid (e.g. B x beta for the memory-speed trade-off, c_p x c_d for pricing)."""
    out = np.zeros((len(v1), len(v2)))
    for a, x in enumerate(v1):
        for b, y in enumerate(v2):
            kw = {p1: int(x) if p1 == "B" else float(x), p2: int(y) if p2 == "B" else float(y)}
            out[a, b] = solve(replace(inst, **kw))[0]
    return out
