"""Pins of the CPU oracle of the exponential-service model (Section 2.3) against what the paper and queueing
theory fix: flow balance Eq. (15)-(20), capacity Eq. (12)-(14), M/M/infinity and birth-death stationary laws,
Poisson arrivals, and the optimality / occupancy-convergence theorems of Sections 4 and 5."""
import numpy as np
import pytest

from oracle import CtmcOracle, ctmc_revenue_rate, run_ctmc_oracle
from qsim_inputs import presets
from qsim_inputs.spec import GATE_PRIORITY, ROUTER_SLI, ROUTER_SOLO_FIRST, CtmcInputs


def one_class(N, M, B, lam, mu_p, mu_m, mu_s, theta, R=6, seed=3, qcap=4096):
    a = lambda v: np.array([v], float)
    inp = CtmcInputs(name="one", I=1, N=N, M=M, B=B, R=R, qcap=qcap, seed=seed, lam=a(lam), theta=a(theta), mu_p=a(mu_p),
                     mu_m=a(mu_m), mu_s=a(mu_s), P=a(100), D=a(100), prices=np.array([1.0, 2.0]),
                     prio_rank=np.zeros(1, np.uint32), xstar=a(0.5), n_xstar=a(0.5 * N), n_qpstar=a(0.0), p_solo=a(1.0))
    inp.validate()
    return inp


def window(inp, T1, T2):
    sim = CtmcOracle(inp)
    sim.run_until(T1); a = sim.stats()
    sim.run_until(T2); b = sim.stats()
    sim.close()
    d = {k: b[k] - a[k] for k in b}
    for k in ("Qp", "X", "Qd", "Ym", "Ys"):
        d[k] = b[k]
        d[k + "_start"] = a[k]
    return d


def check_balance(st, start=None):
    z = lambda k: 0 if start is None else start[k].astype(np.int64)
    g = lambda k: st[k].astype(np.int64)
    # Eq. (15)-(20): every stage's content is what entered minus what left
    assert np.array_equal(g("Qp") - z("Qp"), g("arrivals") - g("admitted") - g("abandoned_p"))
    assert np.array_equal(g("X") - z("X"), g("admitted") - g("prefill_done"))
    assert np.array_equal(g("Qd") - z("Qd"), g("prefill_done") - g("placed_mixed") - g("placed_solo") - g("abandoned_d") - g("overflow_d"))
    assert np.array_equal(g("Ym") + g("Ys") - z("Ym") - z("Ys"), g("placed_mixed") + g("placed_solo") - g("done_mixed") - g("done_solo"))


@pytest.mark.parametrize("router,gate,theta", [(ROUTER_SOLO_FIRST, 0, (0.1, 0.1)), (ROUTER_SLI, 0, (0.1, 0.1)),
                                                (ROUTER_SOLO_FIRST, GATE_PRIORITY, (0.0, 0.3)), (ROUTER_SLI, 0, (0.0, 0.0))])
def test_flow_balance_and_capacity(router, gate, theta):
    # overloaded (1.6x the nominal rates) so that both queues fill and the decode buffers are used
    inp = presets.ctmc_instance(n=12, R=5, router=router, gate=gate, theta=theta, lam=(0.8, 0.8))
    st = run_ctmc_oracle(inp, 150.0)         # the oracle itself returns an error when Eq. (12)-(14) break
    check_balance(st)
    assert (st["X"].sum(1) <= inp.M).all()
    assert (st["Ym"].sum(1) <= inp.M * (inp.B - 1)).all() and (st["Ys"].sum(1) <= (inp.N - inp.M) * inp.B).all()
    assert (st["abandoned_p"].sum() > 0) == (max(theta) > 0)
    if min(theta) > 0:
        assert st["overflow_d"].sum() == 0      # patient classes can fill the bounded buffer under this overload
    assert st["events"].sum() == sum(int(st[k].sum()) for k in ("arrivals", "abandoned_p", "abandoned_d", "prefill_done", "done_mixed", "done_solo"))


def test_resumable_and_replication_keyed():
    inp = presets.ctmc_instance(n=10, R=4, router=ROUTER_SLI)
    whole = run_ctmc_oracle(inp, 80.0)
    sim = CtmcOracle(inp)
    for T in (13.0, 13.0, 41.5, 80.0):
        sim.run_until(T)
    parts = sim.stats(); sim.close()
    for k in whole:
        assert np.array_equal(whole[k], parts[k]), k
    shifted = run_ctmc_oracle(inp.with_(rep_offset=2, R=2), 80.0)
    for k in whole:
        assert np.array_equal(whole[k][2:], shifted[k]), k


def test_infinite_server_stages():
    # no stage ever blocks: prefill and solo decode are M/M/infinity, so the mean contents are rate / mu
    N, lam, mu_p, mu_s = 40, 0.25, 5.0, 0.8
    inp = one_class(N=N, M=20, B=1000, lam=lam, mu_p=mu_p, mu_m=0.3, mu_s=mu_s, theta=0.2, R=8)
    d = window(inp, 50.0, 1050.0)
    T = d["T_elapsed"][0]
    assert d["abandoned_p"].sum() == 0 and d["placed_mixed"].sum() == 0
    X = d["area_X"].sum() / (T * inp.R); Ys = d["area_Ys"].sum() / (T * inp.R)
    # Poisson stationary law: variance of the time average ~ 2 mean / (mu T R)
    assert abs(X - N * lam / mu_p) < 5 * np.sqrt(2 * N * lam / mu_p / (mu_p * T * inp.R))
    assert abs(Ys - N * lam / mu_s) < 5 * np.sqrt(2 * N * lam / mu_s / (mu_s * T * inp.R))
    # all GPUs mixed: the same requests decode at the mixed rate
    inp = one_class(N=N, M=N, B=1000, lam=lam, mu_p=mu_p, mu_m=0.3, mu_s=mu_s, theta=0.2, R=8)
    d = window(inp, 50.0, 1050.0)
    Ym = d["area_Ym"].sum() / (T * inp.R)
    assert d["placed_solo"].sum() == 0
    assert abs(Ym - N * lam / 0.3) < 5 * np.sqrt(2 * N * lam / 0.3 / (0.3 * T * inp.R))


def birth_death(birth, death, kmax=400):
    w = np.ones(kmax)
    for k in range(1, kmax):
        w[k] = w[k - 1] * birth / death(k)
    return w / w.sum()


def test_single_server_prefill_queue_with_abandonment():
    # one GPU, one prefill slot: Q_p + X is the M/M/1+M birth-death chain (birth lambda, death mu_p + (k-1) theta)
    lam, mu_p, theta = 1.5, 1.0, 0.4
    inp = one_class(N=1, M=1, B=10_000, lam=lam, mu_p=mu_p, mu_m=50.0, mu_s=50.0, theta=theta, R=8, seed=9)
    d = window(inp, 100.0, 6100.0)
    pi = birth_death(lam, lambda k: mu_p + (k - 1) * theta)
    k = np.arange(len(pi))
    Qp_mean = float((np.maximum(k - 1, 0) * pi).sum()); X_mean = 1.0 - pi[0]
    T = d["T_elapsed"][0] * inp.R
    assert abs(d["area_Qp"].sum() / T - Qp_mean) < 0.04 * Qp_mean
    assert abs(d["area_X"].sum() / T - X_mean) < 0.02 * X_mean
    # abandonment rate = theta E[Q_p]
    assert abs(d["abandoned_p"].sum() / T - theta * Qp_mean) < 0.05 * theta * Qp_mean


def test_decode_buffer_with_abandonment_is_erlang_a():
    # prefill is almost instantaneous, equal decode speeds in both groups: the decode stage is M/M/5+M
    lam_tot, mu, theta = 4.5, 1.0, 0.5
    inp = one_class(N=4, M=3, B=2, lam=lam_tot / 4, mu_p=2000.0, mu_m=mu, mu_s=mu, theta=theta, R=8, seed=21)
    d = window(inp, 100.0, 4100.0)
    c = 3 * 1 + 1 * 2
    pi = birth_death(lam_tot, lambda k: min(k, c) * mu + max(k - c, 0) * theta)
    k = np.arange(len(pi))
    Qd_mean = float((np.maximum(k - c, 0) * pi).sum())
    T = d["T_elapsed"][0] * inp.R
    assert abs(d["area_Qd"].sum() / T - Qd_mean) < 0.05 * Qd_mean
    assert abs(d["abandoned_d"].sum() / T - theta * Qd_mean) < 0.06 * theta * Qd_mean
    # solo slots are taken first: the solo group is the busier one per slot
    assert d["area_Ys"].sum() / 2 > d["area_Ym"].sum() / 3


def test_poisson_arrivals():
    inp = presets.ctmc_instance(n=30, R=64, lam=(0.5, 0.2))
    st = run_ctmc_oracle(inp, 40.0)
    for i, lam in enumerate((0.5, 0.2)):
        m = 30 * lam * 40.0
        a = st["arrivals"][:, i].astype(float)
        assert abs(a.mean() - m) < 4 * np.sqrt(m / 64)
        assert 0.6 < a.var(ddof=1) / m < 1.5


def test_priority_gate_serves_the_first_rank_under_backlog():
    # overload (every GPU mixed, prefill saturated): the class with the larger D/P (rank 0) is admitted as soon as a
    # prefill slot frees, so it waits for one residual service at most; the other class absorbs the whole backlog
    inp = presets.ctmc_instance(n=20, R=4, gate=GATE_PRIORITY, lam=(3.0, 3.0), theta=(0.05, 0.05))
    st = run_ctmc_oracle(inp, 200.0)
    first = int(np.argmin(inp.prio_rank))
    other = 1 - first
    assert inp.prio_rank[first] == 0 and inp.D[first] / inp.P[first] > inp.D[other] / inp.P[other]
    assert (st["admitted"][:, first] > 0.995 * st["arrivals"][:, first]).all()
    assert (st["abandoned_p"][:, other] > 0.15 * st["arrivals"][:, other]).all()
    assert st["area_Qp"][:, first].mean() < 0.02 * st["area_Qp"][:, other].mean()
    # the occupancy gate holds the same class back once it is above its target, so it queues more than under priority
    occ = run_ctmc_oracle(inp.with_(gate=0), 200.0)
    assert occ["area_Qp"][:, first].mean() > 1.5 * st["area_Qp"][:, first].mean()


def revenue_window(inp, T1, T2):
    d = window(inp, T1, T2)
    return ctmc_revenue_rate(inp, d), d


def test_revenue_converges_to_the_lp_optimum():
    # asymptotic optimality (Sections 4 and 5.1): the per-GPU revenue rate approaches the LP value as n grows
    gaps = []
    for n in (20, 200, 1000):
        inp = presets.ctmc_instance(n=n, R=3)
        rev, _ = revenue_window(inp, 200.0, 600.0)
        gaps.append(1.0 - rev.mean() / inp.meta["lp_value"])
    assert gaps[0] > gaps[1] > gaps[2] > 0.0
    assert gaps[2] < 0.008 and gaps[0] > 0.015


def test_sli_router_occupancies_converge_to_the_plan():
    # Section 5.2: with the randomized router prefill and decode occupancies follow the LP solution class by class
    n = 1000
    inp = presets.ctmc_instance(n=n, R=3, router=ROUTER_SLI)
    rev, d = revenue_window(inp, 200.0, 600.0)
    T = d["T_elapsed"][:, None]
    plan = inp.meta["plan"]
    assert np.allclose((d["area_X"] / T / n).mean(0)[1], plan["x"][1], rtol=0.02)
    assert np.allclose((d["area_Ym"] / T / n).mean(0), plan["ym"], rtol=0.02, atol=1e-9)
    assert np.allclose((d["area_Ys"] / T / n).mean(0), plan["ys"], rtol=0.04)
    assert 1.0 - rev.mean() / inp.meta["lp_value"] < 0.006
