"""Host-side static planning: the steady-state fluid LP and what the policy derives from it.

This is set-up work, done once per block before any simulation starts; its results are
handed to a simulator as plain numbers (M, x*, n x*, n q*_p, p_s).  No simulator imports it.

* service rates                     Eq. (4):  mu_p = C/(P tau), mu_m = 1/(D tau), mu_s = gamma/D
* bundled LP                        Eq. (36)
* separate-charging objective       Eq. (38)
* number of mixed GPUs              M = ceil(n sum_i x*_i)            (Section 4.1, Static Planning)
* solo probability of the SLI router p_s,i                            (Section 5.2, Dynamic control)
* average-TPOT SLI                  Eq. (42)-(43)
* prefill / decode fairness SLIs    Eq. (39), (41)
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
from scipy.optimize import linprog


def iteration_time(coeffs: Sequence[float], p: int, d: int, K: int = 0) -> float:
    """Nominal iteration time of the six-coefficient family (alpha_m, beta, delta_m, alpha_s, delta_s, kappa).

    Used here only to obtain the two constants (tau_mix, tau_solo) the LP needs; simulators
    carry their own implementation with a fixed rounding order.
    """
    am, beta, dm, a_s, ds, kappa = coeffs
    t = am + beta * p + dm * d if p > 0 else a_s + ds * d
    return t + kappa * K


def nominal_taus(coeffs: Sequence[float], B: int, C: int) -> tuple[float, float]:
    """(tau_mix, tau_solo) used for planning: a full mixed batch and a full solo batch."""
    return iteration_time(coeffs, C, B - 1), iteration_time(coeffs, 0, B)


def service_rates(P, D, C: int, tau_mix: float, tau_solo: float, beta=None, nchunks=None):
    """Eq. (4).  With `nchunks` (mean number of prefill iterations per request, E ceil(P/C)) and the
    per-token slope `beta`, the prefill rate accounts for chunking: a request then spends
    nchunks * (tau_mix - beta C) + beta P in prefill, which equals (P/C) tau_mix when P is a multiple of C."""
    P = np.asarray(P, float)
    D = np.asarray(D, float)
    if nchunks is None:
        mu_p = C / (P * tau_mix)
    else:
        mu_p = 1.0 / (np.asarray(nchunks, float) * (tau_mix - beta * C) + beta * P)
    mu_m = 1.0 / (D * tau_mix)
    mu_s = (1.0 / tau_solo) / D
    return mu_p, mu_m, mu_s


def consistent_taus(coeffs, B: int, C: int, solve, iters: int = 40, tol: float = 1e-10, start=None):
    """Planning constants (tau_mix, tau_solo) when the iteration time depends on the decode count.

    The paper's law (Eq. (2)-(3)) has constant tau_mix and tau_solo; with a per-decode slope the LP needs
    the batch sizes it induces.  Fixed point: solve the LP under the current constants (`solve` maps
    (tau_mix, tau_solo) to a Plan), read the mean decodes per mixed GPU  sum y_m / sum x  and per solo GPU
    sum y_s / (1 - sum x), and re-evaluate tau there.  Starts from full batches, which is exact when
    the slopes are zero (or from `start`).  Returns (tau_mix, tau_solo, plan).
    """
    tm, ts = start if start is not None else nominal_taus(coeffs, B, C)
    plan = solve(tm, ts)
    if coeffs[2] == 0.0 and coeffs[4] == 0.0:
        return tm, ts, plan
    for _ in range(iters):
        X = float(plan.x.sum())
        d_m = float(plan.ym.sum()) / X if X > 1e-12 else 0.0
        d_s = float(plan.ys.sum()) / (1.0 - X) if 1.0 - X > 1e-12 else float(B)
        d_m = min(max(d_m, 0.0), B - 1)
        d_s = min(max(d_s, 1.0), B)
        # damped update keeps the iteration from oscillating between vertex solutions
        tm_new = 0.5 * tm + 0.5 * (coeffs[0] + coeffs[1] * C + coeffs[2] * d_m)
        ts_new = 0.5 * ts + 0.5 * (coeffs[3] + coeffs[4] * d_s)
        done = abs(tm_new - tm) < tol and abs(ts_new - ts) < tol
        tm, ts = tm_new, ts_new
        plan = solve(tm, ts)
        if done:
            break
    return tm, ts, plan


def fluid_capacity(pi, P, D, B: int, C: int, tau_mix: float, tau_solo: float, beta=None, nchunks=None) -> float:
    """Largest total per-GPU arrival rate s such that lambda = s*pi is servable with empty queues.

    From the capacity and flow-balance rows of Eq. (36) with theta = 0, q = 0:
    x = s*b with b = (tau/C) sum pi_i P_i (prefill capacity: x <= 1), and decode work
    s*a with a = tau sum pi_i D_i measured in mixed-slot time must fit
    y_m + y_s/kappa' ... which gives s <= kB / (a + (kB - (B-1)) b), k = tau_mix/tau_solo.
    """
    pi = np.asarray(pi, float)
    mu_p, _, _ = service_rates(P, D, C, tau_mix, tau_solo, beta, nchunks)
    a = tau_mix * float(np.dot(pi, D))
    b = float(np.sum(pi / mu_p))
    k = tau_mix / tau_solo
    return min(1.0 / b, k * B / (a + (k * B - (B - 1)) * b))


@dataclass
class Plan:
    x: np.ndarray
    ym: np.ndarray
    ys: np.ndarray
    qp: np.ndarray
    qd: np.ndarray
    value: float          # LP optimum (per-GPU reward rate of the chosen objective)
    tau_mix: float
    tau_solo: float

    def M(self, n: int) -> int:
        # small slack so that an exactly-integer n*sum(x*) is not pushed up by LP round-off
        return int(min(n, max(0, math.ceil(n * float(self.x.sum()) - 1e-9))))

    def p_solo(self, mu_m, mu_s) -> np.ndarray:
        num = mu_s * self.ys
        den = mu_m * self.ym + num
        out = np.ones_like(num)
        nz = den > 0
        out[nz] = num[nz] / den[nz]
        return np.clip(out, 0.0, 1.0)


def pool_weights(plan: "Plan", mu_m, mu_s):
    """Class-selection weights of the general SLI-aware router: varpi_m,i = mu_m y*_m,i / sum_j mu_m,j y*_m,j and
    the same for the solo pool (0/0 := 0)."""
    wm = mu_m * plan.ym
    ws = mu_s * plan.ys
    wm = wm / wm.sum() if wm.sum() > 0 else np.zeros_like(wm)
    ws = ws / ws.sum() if ws.sum() > 0 else np.zeros_like(ws)
    return ws, wm


def solve_plan(lam, P, D, theta, B: int, C: int, tau_mix: float, tau_solo: float,
               c_p: float, c_d: float, separate: bool = False,
               qd_zero: bool = False,
               tpot_cap: Optional[float] = None,
               prefill_fair: Optional[float] = None,
               decode_fair: Optional[float] = None,
               min_admit_ratio: Optional[float] = None,
               max_prefill_wait: Optional[float] = None,
               beta=None, nchunks=None) -> Plan:
    """Solve Eq. (36) (or its Eq. (38) objective) with optional SLI rows.

    Variable order: x[0:I], ym[I:2I], ys[2I:3I], qp[3I:4I], qd[4I:5I].
    A class with theta_i = 0 cannot hold fluid queue mass in steady state; its prefill balance
    becomes mu_p x_i <= lambda_i (the theta -> 0+ limit) and q_p,i = q_d,i = 0.
    `min_admit_ratio` (mu_p x_i >= r lambda_i) and `max_prefill_wait`
    (q_p,i <= (w - P_i tau / C) mu_p x_i, a Little's-law mean-wait proxy) are linear stand-ins
    for an admission-ratio floor and a time-to-first-token cap; they are not SLIs of the paper.
    """
    lam = np.asarray(lam, float)
    P = np.asarray(P, float)
    D = np.asarray(D, float)
    theta = np.asarray(theta, float)
    I = len(lam)
    mu_p, mu_m, mu_s = service_rates(P, D, C, tau_mix, tau_solo, beta, nchunks)
    nv = 5 * I
    ix, iym, iys, iqp, iqd = (slice(k * I, (k + 1) * I) for k in range(5))

    c = np.zeros(nv)
    if separate:
        c[ix] = c_p * P * mu_p          # = c_p C / tau_mix under Eq. (4)
        c[iym] = c_d / tau_mix
        c[iys] = c_d / tau_solo
    else:
        w = c_p * P + c_d * D
        c[iym] = w * mu_m
        c[iys] = w * mu_s

    A_ub, b_ub, A_eq, b_eq = [], [], [], []

    def row():
        return np.zeros(nv)

    r = row(); r[ix] = 1.0; A_ub.append(r); b_ub.append(1.0)                       # prefill capacity
    r = row(); r[iym] = 1.0; r[ix] = -(B - 1); A_ub.append(r); b_ub.append(0.0)    # mixed decode capacity
    r = row(); r[iys] = 1.0; r[ix] = B; A_ub.append(r); b_ub.append(float(B))      # solo decode capacity
    for i in range(I):
        r = row(); r[ix.start + i] = mu_p[i]
        if theta[i] > 0:
            r[iqp.start + i] = theta[i]; A_eq.append(r); b_eq.append(lam[i])       # prefill flow balance
        else:
            A_ub.append(r); b_ub.append(lam[i])
        r = row()                                                                   # decode flow balance
        r[ix.start + i] = mu_p[i]; r[iqd.start + i] = -theta[i]
        r[iym.start + i] = -mu_m[i]; r[iys.start + i] = -mu_s[i]
        A_eq.append(r); b_eq.append(0.0)
    bounds = [(0, None)] * nv
    for i in range(I):
        if theta[i] <= 0:
            bounds[iqp.start + i] = (0, 0)
            bounds[iqd.start + i] = (0, 0)
        if qd_zero:
            bounds[iqd.start + i] = (0, 0)
    if tpot_cap is not None:
        # Eq. (42) multiplied out: (tau(B-1) - B/gamma - eta((B-1) - B)) X <= eta B - B/gamma
        r = row(); r[ix] = tau_mix * (B - 1) - tau_solo * B + tpot_cap
        A_ub.append(r); b_ub.append(tpot_cap * B - tau_solo * B)
    for fair, sl in ((prefill_fair, ix), (decode_fair, iys)):
        if fair is not None:
            for i in range(I):
                for j in range(I):
                    if i != j:
                        r = row(); r[sl.start + i] = 1.0; r[sl.start + j] = -1.0
                        A_ub.append(r); b_ub.append(fair)
    if min_admit_ratio is not None:
        for i in range(I):
            r = row(); r[ix.start + i] = -mu_p[i]; A_ub.append(r); b_ub.append(-min_admit_ratio * lam[i])
    if max_prefill_wait is not None:
        for i in range(I):
            slack = max(max_prefill_wait - 1.0 / mu_p[i], 0.0)
            r = row(); r[iqp.start + i] = 1.0; r[ix.start + i] = -slack * mu_p[i]
            A_ub.append(r); b_ub.append(0.0)

    res = linprog(-c, A_ub=np.array(A_ub), b_ub=np.array(b_ub),
                  A_eq=np.array(A_eq) if A_eq else None, b_eq=np.array(b_eq) if b_eq else None,
                  bounds=bounds, method="highs")
    if res.status != 0:
        raise RuntimeError(f"fluid LP failed: {res.message}")
    z = np.maximum(res.x, 0.0)
    return Plan(x=z[ix].copy(), ym=z[iym].copy(), ys=z[iys].copy(), qp=z[iqp].copy(), qd=z[iqd].copy(),
                value=float(-res.fun), tau_mix=tau_mix, tau_solo=tau_solo)


def priority_ranks(P, D) -> np.ndarray:
    """Static ranks of the Prioritize-and-Route gate: rank 0 = largest D_i/P_i; ties keep index order."""
    ratio = np.asarray(D, float) / np.asarray(P, float)
    order = sorted(range(len(ratio)), key=lambda i: (-ratio[i], i))
    ranks = np.zeros(len(ratio), np.uint32)
    for r, i in enumerate(order):
        ranks[i] = r
    return ranks
