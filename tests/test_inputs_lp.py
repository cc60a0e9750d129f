"""Host-side planning against closed forms the paper fixes."""
import math

import numpy as np

from qsim_inputs import fluid_lp as lp
from qsim_inputs import presets


def test_service_rates_eq4():
    mu_p, mu_m, mu_s = lp.service_rates([300, 3000], [1000, 400], 256, 0.033272, 0.022)
    assert np.allclose(mu_p, [256 / (300 * 0.033272), 256 / (3000 * 0.033272)])
    assert np.allclose(mu_m, [1 / (1000 * 0.033272), 1 / (400 * 0.033272)])
    assert np.allclose(mu_s, [(1 / 0.022) / 1000, (1 / 0.022) / 400])
    # mu_m / mu_s = 1 / (gamma tau) for every class (proof of Proposition 1)
    assert np.allclose(mu_m / mu_s, 0.022 / 0.033272)


def test_lp_value_equals_offered_revenue_when_underloaded_and_capacity_is_tight():
    P, D, B, C = [256, 1024], [64, 256], 32, 256
    tm, ts = lp.nominal_taus(presets.COEFFS_BENCH, B, C)
    pi = np.array([0.5, 0.5])
    s = lp.fluid_capacity(pi, P, D, B, C, tm, ts)
    w = 1.0 * np.array(P) + 2.0 * np.array(D)
    for load in (0.5, 0.9, 1.0):
        plan = lp.solve_plan(load * s * pi, P, D, [0, 0], B, C, tm, ts, 1.0, 2.0)
        assert math.isclose(plan.value, float(np.dot(load * s * pi, w)), rel_tol=1e-7)
    # just above capacity with patience the LP can no longer serve everything
    over = lp.solve_plan(1.05 * s * pi, P, D, [0.1, 0.1], B, C, tm, ts, 1.0, 2.0)
    assert over.value < float(np.dot(1.05 * s * pi, w)) * (1 - 1e-4)
    assert over.value >= float(np.dot(s * pi, w)) * (1 - 1e-7)
    # capacity rows of Eq. (36) hold
    for plan in (over,):
        X = plan.x.sum()
        assert X <= 1 + 1e-9 and plan.ym.sum() <= (B - 1) * X + 1e-7 and plan.ys.sum() <= B * (1 - X) + 1e-7


def test_proposition_1_decode_buffer_elimination():
    # gamma tau >= (B-1)/B  =>  an optimal solution with q_d = 0 exists: forcing q_d = 0 costs nothing
    P, D, B, C = [300, 3000], [1000, 400], 16, 256
    tm, ts = 0.033272, 0.022
    assert (1 / ts) * tm >= (B - 1) / B
    for lam in ([0.5, 0.5], [0.3, 0.6], [1.0, 0.2]):
        free = lp.solve_plan(lam, P, D, [0.1, 0.1], B, C, tm, ts, 0.1, 0.2)
        forced = lp.solve_plan(lam, P, D, [0.1, 0.1], B, C, tm, ts, 0.1, 0.2, qd_zero=True)
        assert math.isclose(free.value, forced.value, rel_tol=1e-8)


def test_separate_objective_depends_on_aggregates_only():
    # Eq. (38): value = c_p C/tau sum x + c_d/tau sum y_m + c_d gamma sum y_s
    P, D, B, C = [300, 3000], [1000, 400], 16, 256
    tm, ts = 0.033272, 0.022
    plan = lp.solve_plan([0.5, 0.5], P, D, [0.1, 0.1], B, C, tm, ts, 0.1, 0.2, separate=True)
    v = 0.1 * C / tm * plan.x.sum() + 0.2 / tm * plan.ym.sum() + 0.2 / ts * plan.ys.sum()
    assert math.isclose(plan.value, v, rel_tol=1e-9)
    # the per-class form of the same objective (Eq. (23) in fluid form) gives the same number
    mu_p, mu_m, mu_s = lp.service_rates(P, D, C, tm, ts)
    v2 = float(np.sum(0.1 * np.array(P) * mu_p * plan.x + 0.2 * np.array(D) * (mu_m * plan.ym + mu_s * plan.ys)))
    assert math.isclose(v, v2, rel_tol=1e-9)


def test_tpot_cap_binds():
    P, D, B, C = [300, 3000], [1000, 400], 16, 256
    tm, ts = 0.033272, 0.022
    free = lp.solve_plan([0.5, 0.5], P, D, [0.1, 0.1], B, C, tm, ts, 0.1, 0.2)
    X = free.x.sum()
    tpot = (tm * (B - 1) * X + ts * B * (1 - X)) / ((B - 1) * X + B * (1 - X))     # Eq. (42)
    capped = lp.solve_plan([0.5, 0.5], P, D, [0.1, 0.1], B, C, tm, ts, 0.1, 0.2, tpot_cap=0.9 * tpot + 0.1 * ts)
    Xc = capped.x.sum()
    tpot_c = (tm * (B - 1) * Xc + ts * B * (1 - Xc)) / ((B - 1) * Xc + B * (1 - Xc))
    assert tpot_c <= 0.9 * tpot + 0.1 * ts + 1e-9 and capped.value < free.value


def test_mixed_gpu_count_and_priority_ranks():
    plan = lp.Plan(x=np.array([0.1, 0.15]), ym=np.zeros(2), ys=np.zeros(2), qp=np.zeros(2), qd=np.zeros(2),
                   value=0.0, tau_mix=1.0, tau_solo=1.0)
    assert plan.M(10) == 3 and plan.M(100) == 25 and plan.M(4) == 1      # M = ceil(n sum x*)
    assert list(lp.priority_ranks([300, 3000], [1000, 400])) == [0, 1]   # D/P: 3.33 > 0.13
    assert list(lp.priority_ranks([100, 100, 50], [10, 20, 10])) == [2, 0, 1]


def test_recipes_are_deterministic_and_valid():
    a, b = presets.cfg1(R=2), presets.cfg1(R=2)
    assert np.array_equal(a.lengths, b.lengths) and np.array_equal(a.xstar, b.xstar) and a.M[0] == b.M[0]
    for inp in (presets.cfg0(), presets.cfg2(N=32, R=2), presets.cfg3(N=32, R=2, block_len=5.0),
                presets.cfg4(N=32, R=2), presets.paper_instance()):
        inp.validate()
        assert np.all(inp.M <= inp.N) and np.all(inp.xstar >= 0) and np.all((inp.p_solo >= 0) & (inp.p_solo <= 1))
    c3 = presets.cfg3(N=32, R=2, block_len=5.0)
    assert c3.nblk == 24 and c3.rates.shape == (24, 4)
    # sinusoid of amplitude 0.5 around 0.95 of capacity
    tot = c3.rates.sum(axis=1) / c3.meta["capacity"]
    assert math.isclose(tot.max(), 1.45, rel_tol=1e-9) and math.isclose(tot.min(), 0.45, rel_tol=1e-9)


def test_planning_grids_show_what_the_paper_reports_for_them():
    """Section 6.3 (figures only, so the pins are the trends the text states): prefill fairness is dear and decode
    fairness cheap; the price of a TPOT target explodes towards the floor 1/gamma = 0.022 s and no plan exists below it;
    revenue grows with B and saturates around B = 16; it falls with beta and alpha and rises with gamma."""
    from qsim_inputs import lp_sweeps as S
    inst = S.Instance()
    free, plan = S.solve(inst, qd_zero=True)
    pf = S.frontier(inst, "prefill_fair", [0.0, 0.05, 0.1, 0.2, 1.0])
    df = S.frontier(inst, "decode_fair", [0.0, 1.0, 2.0, 4.0, 16.0])
    assert np.all(np.diff(pf) >= -1e-9) and np.all(np.diff(df) >= -1e-9)          # a looser target never costs revenue
    assert abs(pf[-1] - free) < 1e-6 and abs(df[-1] - free) < 1e-6              # and a slack one costs nothing
    assert (free - pf[0]) > 3.0 * (free - df[0]) and pf[0] < 0.5 * free           # prefill fairness: steep; decode fairness: mild
    etas = [0.0215, 0.02205, 0.0221, 0.0225, 0.023, 0.024, 0.026, 0.030]
    tp = S.frontier(inst, "tpot_cap", etas)
    assert np.isnan(tp[0]) and np.all(np.isfinite(tp[1:]))                        # nothing is feasible below 1/gamma
    price = S.shadow_price(etas[1:], tp[1:])
    assert np.all(np.diff(price) <= 1e-6) and price[0] > 5.0 * price[-3] > 0.0 and price[0] > 50.0 * price[-2] > 0.0   # marginal revenue per second of TPOT: steepest at the floor
    assert abs(tp[-1] - free) < 1e-6
    # the TPOT target is met with equality while it binds (Eq. (43))
    _, p2 = S.solve(inst, qd_zero=True, tpot_cap=0.023)
    assert abs(S.average_tpot(inst, float(p2.x.sum())) - 0.023) < 1e-9
    rev_B, tpot_B = S.sensitivity(inst, "B", [2, 4, 8, 16, 32, 64])
    assert np.all(np.diff(rev_B) >= -1e-9) and rev_B[3] > 0.97 * rev_B[-1] and rev_B[1] < 0.7 * rev_B[-1] and rev_B[-2] == rev_B[-1]
    rev_b, tpot_b = S.sensitivity(inst, "beta", [1e-5, 6.2e-5, 3e-4, 1e-3])
    assert np.all(np.diff(rev_b) <= 1e-9) and rev_b[-1] < 0.5 * rev_b[0] and np.all(np.diff(tpot_b) > 0)
    rev_a, _ = S.sensitivity(inst, "alpha", [0.02, 0.05, 0.1, 0.15])
    assert np.all(np.diff(rev_a) < 0)
    rev_g, tpot_g = S.sensitivity(inst, "gamma", [10.0, 20.0, 30.0, 45.0])
    assert np.all(np.diff(rev_g) > 0) and np.all(np.diff(tpot_g) < 0)
    # the memory-speed grid: more slots help, slower prefill hurts, everywhere
    g = S.grid(inst, "B", [4, 8, 16, 32], "beta", [3e-5, 6.2e-5, 2e-4])
    assert np.all(np.diff(g, axis=0) >= -1e-9) and np.all(np.diff(g, axis=1) <= 1e-9)
