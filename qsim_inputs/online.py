"""Online adaptive controller of the trace-replay experiment (Section 6.2): rolling-window rate estimate,
periodic re-solve of the fluid LP, new mixed/solo split.  Host-side; drives any simulator object that offers
run_until(T), stats() and set_targets(M, x*, n x*, n q*_p, p_s)."""
from __future__ import annotations

import numpy as np

from . import fluid_lp as lp


def estimate_rates(A_now, A_past, n: int, t_k: float, W: float = 30.0, rho: float = 3.0, lam_min: float = 1e-6,
                   eps: float = 1e-9):
    """Eq. (45): lambda_hat_i = max{ rho N_i / (n W_bar), lambda_min }, N_i arrivals in the last window,
    W_bar = min{W, max{t_k, eps}}."""
    Wbar = min(W, max(t_k, eps))
    N = np.asarray(A_now, float) - np.asarray(A_past, float)
    return np.maximum(rho * N / (n * Wbar), lam_min)


def replan(lam_hat, Pm, Dm, n: int, B: int, C: int, coeffs, prices, separate: bool, theta: float = 3e-4):
    """Re-solve the planning LP with the estimated rates (common small impatience theta keeps it well posed)
    and return (M, x*, n x*, n q*_p, p_s); M follows Eq. (46)."""
    I = len(lam_hat)
    th = np.full(I, theta)

    def solve(tm, ts):
        return lp.solve_plan(lam_hat, Pm, Dm, th, B, C, tm, ts, prices[0], prices[1], separate=separate)

    tm, ts, plan = lp.consistent_taus(coeffs, B, C, solve)
    _, mu_m, mu_s = lp.service_rates(Pm, Dm, C, tm, ts)
    return plan.M(n), plan.x, n * plan.x, n * plan.qp, plan.p_solo(mu_m, mu_s)


def run_online(sim, inp, Pm, Dm, T_total: float, period: float = 10.0, W: float = 30.0, rho: float = 3.0):
    """Drive `sim` to T_total with replanning every `period` seconds.  Arrival counts are read from replication 0
    (trace replay feeds every replication the same arrivals).  Returns the list of (t_k, M) decisions."""
    history = {0.0: np.zeros(inp.I)}
    decisions = []
    k = 0
    while True:
        t_k = k * period
        if t_k >= T_total:
            break
        if k > 0:
            sim.run_until(t_k)
            history[t_k] = sim.stats()["arrivals"][0].astype(float)
            t_past = max(t_k - W, 0.0)
            past = history[min(history, key=lambda x: abs(x - t_past))]
            lam_hat = estimate_rates(history[t_k], past, inp.N, t_k, W=W, rho=rho)
            M, xs, nx, nq, ps = replan(lam_hat, Pm, Dm, inp.N, inp.B, inp.C, inp.coeffs, inp.prices,
                                       separate=inp.pricing == 1)
            sim.set_targets(M, xs, nx, nq, ps)
            decisions.append((t_k, int(M)))
        k += 1
    sim.run_until(T_total)
    return decisions
