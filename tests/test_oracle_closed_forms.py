"""Closed forms and limit statements the oracle must reproduce."""
import math

import numpy as np
import pytest

from oracle import OracleSim, run_oracle
from qsim_inputs import presets
from qsim_inputs.spec import ROUTER_SLI


def band(x, k=5.0):
    x = np.asarray(x, float)
    return k * x.std(ddof=1) / math.sqrt(x.size)


def test_arrivals_are_poisson_with_rate_n_lambda():
    # Section 2.3: class-i arrivals are Poisson with rate n * lambda_i.
    inp = presets.cfg0(R=400, horizon_iters=300)
    st = run_oracle(inp, 300)
    T = st["T_elapsed"][0]
    for i in range(inp.I):
        mean = inp.N * inp.rates[0, i] * T
        a = st["arrivals"][:, i].astype(float)
        assert abs(a.mean() - mean) < 5.0 * math.sqrt(mean / a.size)
        # Poisson: variance = mean (dispersion index 1); sd of a sample variance ~ sqrt(2/(R-1)) * var
        assert abs(a.var(ddof=1) / mean - 1.0) < 5.0 * math.sqrt(2.0 / (a.size - 1))


def test_piecewise_constant_rates_follow_the_block_table():
    # rate table switched at block ends: expected count = sum_b n lambda_b,i * block_len
    inp = presets.cfg3(N=4, R=300, block_len=1.5, nblk=6)
    H = int(math.ceil(6 * 1.5 / inp.meta["tau_ref"]))
    st = run_oracle(inp, H)
    T = st["T_elapsed"][0]
    assert T >= 9.0
    for i in range(inp.I):
        mean = sum(inp.N * inp.rates[b, i] * 1.5 for b in range(5)) + inp.N * inp.rates[5, i] * (T - 7.5)
        a = st["arrivals"][:, i].astype(float)
        assert abs(a.mean() - mean) < 5.0 * math.sqrt(mean / a.size)


def test_blocked_class_queue_is_m_m_infinity():
    # A class whose target x* is 0 is never admitted; with exponential patience theta its queue is an
    # M/M/inf system: E Q(t) = (L/theta)(1 - exp(-theta t)), abandonments = arrivals - Q  (Eq. (8)).
    base = presets.single_class(N=2, B=4, P=256, D=4, lam=3.0, theta=0.5, R=600)
    inp = base.with_(xstar=np.zeros((1, 1)), n_xstar=np.zeros((1, 1)))
    tau_ref = inp.meta["tau_ref"]
    H = int(12.0 / tau_ref)
    st = run_oracle(inp, H)
    T = st["T_elapsed"][0]
    Lam, th = 2 * 3.0, 0.5
    assert st["admitted"].sum() == 0
    EQ_T = Lam / th * (1 - math.exp(-th * T))
    area = Lam / th * (T - (1 - math.exp(-th * T)) / th)
    q = st["Qp"][:, 0].astype(float)
    assert abs(q.mean() - EQ_T) < band(q)
    # Poisson marginal: variance = mean
    assert abs(q.var(ddof=1) / EQ_T - 1.0) < 5.0 * math.sqrt(2.0 / (q.size - 1))
    assert abs(st["area_Qp"][:, 0].mean() - area) < band(st["area_Qp"][:, 0])
    ab = st["abandoned_p"][:, 0].astype(float)
    assert abs(ab.mean() - (Lam * T - EQ_T)) < band(ab)
    assert np.array_equal(st["arrivals"][:, 0], st["abandoned_p"][:, 0] + st["Qp"][:, 0])


def test_decode_buffer_abandonment_balances_the_prefill_output():
    # B = 1 on mixed-only GPUs leaves no decode slot (cap B-1 = 0): every finished prefill waits in the
    # decode buffer and leaves by impatience; in steady state E Q_d = throughput / theta  (Eq. (9), (17)).
    inp = presets.single_class(N=3, B=1, P=256, D=4, lam=4.0, theta=2.0, R=300, M=3)
    H = int(20.0 / inp.meta["tau_ref"])
    sim = OracleSim(inp)
    sim.run(H // 4); sim.reset_stats(); sim.run(H)
    st = sim.stats()
    T = st["T_elapsed"][0]
    qd = st["area_Qd"][:, 0] / T
    thr = st["prefill_done"][:, 0] / T
    assert abs(qd.mean() - thr.mean() / 2.0) < band(qd) + band(thr)
    assert st["placed_mixed"].sum() == 0 and st["placed_solo"].sum() == 0
    assert abs(st["abandoned_d"][:, 0].mean() / T - thr.mean()) < band(st["abandoned_d"][:, 0] / T) + band(thr)


def test_no_contention_single_class_closed_form():
    # Requests far apart on one GPU never overlap: TTFT = full chunks * tau(C,0) + tau(last chunk,0),
    # TPOT = tau(0,1), exactly (Eq. (1)-(4) with one request in the system).
    P, D, C = 700, 5, 256
    inj = [(0.5 * k, 0, P, D) for k in range(40)]
    inp = presets.single_class(N=1, B=4, C=C, P=P, D=D, M=1, inject=inj)
    st = run_oracle(inp, int(25.0 / inp.meta["tau_ref"]))
    tau = lambda p, d: 0.005 + 2e-5 * p + 5e-5 * d
    ttft = 2 * tau(256, 0) + tau(700 - 512, 0)
    assert st["done_mixed"][0, 0] == 40
    assert abs(st["sum_ttft"][0, 0] - 40 * ttft) < 1e-10
    assert abs(st["sum_tpot"][0, 0] - 40 * tau(0, 1)) < 1e-10
    assert int(st["iters_mixed"][0]) == 40 * 3 and int(st["iters_solo"][0]) == 40 * D
    assert abs(st["busy_mixed"][0] - 40 * ttft) < 1e-10
    assert abs(st["busy_solo"][0] - 40 * D * tau(0, 1)) < 1e-10


def test_underloaded_cluster_serves_everything():
    # far below capacity: throughput = n lambda, revenue rate per GPU -> lambda (c_p P + c_d D)  (Eq. (22))
    inp = presets.single_class(N=8, B=8, P=512, D=16, lam=2.0, R=40, M=4)
    H = int(200.0 / inp.meta["tau_ref"])
    st = run_oracle(inp, H)
    T = st["T_elapsed"][0]
    rev = (1.0 * st["tokens_in_completed"][:, 0] + 2.0 * st["tokens_out_completed"][:, 0]) / (8 * T)
    assert abs(rev.mean() - 2.0 * (512 + 32)) < band(rev) + 2.0 * (512 + 32) * 0.002
    assert st["abandoned_p"].sum() == 0 and st["Qp"].max() <= 3
    # Little: mean number in prefill = n lambda * prefill time; prefill time is two iterations of tau(256, d)
    x = st["area_X"][:, 0] / T
    lo, hi = 16.0 * 2 * (0.005 + 2e-5 * 256), 16.0 * 2 * (0.005 + 2e-5 * 256 + 5e-5 * 7)
    assert lo - band(x) <= x.mean() <= hi + band(x)


@pytest.mark.parametrize("router", [0, ROUTER_SLI])
def test_revenue_converges_to_the_lp_optimum_as_n_grows(router):
    # Theorems 2-4: per-GPU revenue under gate-and-route approaches the fluid LP optimum and the
    # spread across seeds narrows as n grows.
    gaps, spreads = [], []
    for n, R in ((5, 8), (20, 6), (80, 4)):
        inp = presets.aligned_instance(n=n, R=R, router=router)
        sim = OracleSim(inp)
        sim.run(8000); sim.reset_stats(); sim.run(30000 if n < 80 else 16000)
        st = sim.stats()
        T = st["T_elapsed"]
        rev = (0.1 * st["tokens_in_prefilled"].sum(axis=1) + 0.2 * st["tokens_out_completed"].sum(axis=1)) / (n * T)
        lp = inp.meta["lp_value"][0]
        gaps.append((lp - rev.mean()) / lp)
        spreads.append(rev.std(ddof=1))
        # prefill occupancy tracks the LP target: X_i / n -> x*_i
        if n >= 20:
            x = (st["area_X"] / (n * T[:, None])).mean(axis=0)
            assert np.allclose(x, inp.xstar[0], atol=0.006)
        sim.close()
    assert gaps[0] > gaps[-1] and 0.0 <= gaps[-1] < 0.015
    assert gaps[0] < 0.12
    assert spreads[-1] < spreads[0]


def test_sli_router_tracks_the_decode_split():
    # Theorem 4: under the randomized router Y_m,i/n and Y_s,i/n approach y*_m,i and y*_s,i.
    n = 80
    inp = presets.aligned_instance(n=n, R=3, router=ROUTER_SLI)
    sim = OracleSim(inp)
    sim.run(10000); sim.reset_stats(); sim.run(24000)
    st = sim.stats()
    T = st["T_elapsed"][:, None]
    plan = inp.meta["plan"][0]
    ym = (st["area_Ym"] / (n * T)).mean(axis=0)
    ys = (st["area_Ys"] / (n * T)).mean(axis=0)
    assert np.allclose(ys, plan["ys"], rtol=0.08, atol=0.15)
    assert np.allclose(ym, plan["ym"], rtol=0.08, atol=0.15)
    # class 1 is routed to solo with probability one
    assert inp.p_solo[0, 1] == 1.0 and st["placed_mixed"][:, 1].sum() == 0
    # pool split frequency of class 0 matches p_s,0
    frac = st["placed_solo"][:, 0].sum() / (st["placed_solo"][:, 0].sum() + st["placed_mixed"][:, 0].sum())
    assert abs(frac - inp.p_solo[0, 0]) < 0.02
    sim.close()
