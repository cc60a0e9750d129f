"""Seeded synthetic workload recipes.

Each function returns a `SimInputs` whose LP targets were planned on the host.  The five
`cfg*` recipes are the benchmark configurations (synthetic stand-ins for the production
traces the paper replays, which are not redistributable); `paper_instance` is the synthetic
two-class experiment of the paper's convergence study (Section EC "Convergence Analysis").
"""
from __future__ import annotations

import functools
import math

import numpy as np

from . import fluid_lp as lp
from .lengths import lognormal_tables, table_mean, table_mean_chunks
from .spec import (GATE_FCFS, GATE_OCCUPANCY, GATE_PRIORITY, LENGTH_FIXED, LENGTH_TABLE, PLACE_LEAST_LOADED,
                   PLACE_RANDOM, PRICING_BUNDLED, PRICING_SEPARATE, ROUTER_IMMEDIATE, ROUTER_SLI, ROUTER_SOLO_FIRST,
                   CtmcInputs, SimInputs)

# alpha_m, beta, delta_m, alpha_s, delta_s, kappa
# benchmark family: tau = 5 ms + 0.02 ms * prefill_tokens + 0.05 ms * decode_count
COEFFS_BENCH = np.array([5e-3, 2e-5, 5e-5, 5e-3, 5e-5, 0.0])
# paper calibration (Section 6.1): tau_mix(C) = 0.0174 + 6.2e-5 C; solo iteration 0.022 s
# (the decode-only floor quoted in the SLI study); no dependence on the decode count.
COEFFS_PAPER = np.array([0.0174, 6.2e-5, 0.0, 0.022, 0.0, 0.0])
# paper trace-replay refinement: solo intercept 0.0089 s plus 1.08e-7 s per resident KV token
COEFFS_PAPER_KV = np.array([0.0174, 6.2e-5, 0.0, 0.0089, 0.0, 1.08e-7])


def tau_ref(coeffs, B: int) -> float:
    """Duration of a full solo iteration; a horizon of H iterations means H * tau_ref seconds."""
    return lp.iteration_time(coeffs, 0, B)


def _next_pow2(v: float) -> int:
    return 1 << max(0, int(math.ceil(math.log2(max(v, 1.0)))))


def _plan_block(lam, Pm, Dm, theta, N, B, C, coeffs, prices, separate, nchunks=None, **sli):
    ck = dict(beta=float(coeffs[1]), nchunks=nchunks) if nchunks is not None else {}

    def solve(tm, ts):
        return lp.solve_plan(lam, Pm, Dm, theta, B, C, tm, ts, prices[0], prices[1], separate=separate, **sli, **ck)

    start = None
    if sli:
        # SLI rows can be infeasible under the slow full-batch constants: settle the constants on the
        # unconstrained plan first, then iterate with the constraints
        def relaxed(tm, ts):
            return lp.solve_plan(lam, Pm, Dm, theta, B, C, tm, ts, prices[0], prices[1], separate=separate, **ck)
        tm0, ts0, _ = lp.consistent_taus(coeffs, B, C, relaxed)
        start = (tm0, ts0)
    tau_mix, tau_solo, plan = lp.consistent_taus(coeffs, B, C, solve, start=start)
    _, mu_m, mu_s = lp.service_rates(Pm, Dm, C, tau_mix, tau_solo, **ck)
    return plan, plan.M(N), plan.p_solo(mu_m, mu_s), lp.pool_weights(plan, mu_m, mu_s)


def build(name, *, N, R, B, C, Pm, Dm, lam_blocks, theta, prices, coeffs, gate, router, placement,
          pricing, lengths=None, P_fixed=None, D_fixed=None, seed=0, hist=0, block_len=0.0,
          qcap=None, sli=None, horizon_iters=0, nchunks=None) -> SimInputs:
    """Plan every block and assemble a SimInputs.  Pm/Dm are the class mean lengths the LP uses; nchunks
    (mean prefill iterations per request) makes the planned prefill rate chunk-aware."""
    lam_blocks = np.atleast_2d(np.asarray(lam_blocks, float))
    nblk, I = lam_blocks.shape
    theta = np.asarray(theta, float)
    sli = sli or {}
    M = np.zeros(nblk, np.uint32)
    xs = np.zeros((nblk, I)); nx = np.zeros((nblk, I)); nq = np.zeros((nblk, I)); ps = np.zeros((nblk, I))
    wso = np.zeros((nblk, I)); wmi = np.zeros((nblk, I))
    values, plans = [], []
    for b in range(nblk):
        plan, Mb, p_solo, (w_s, w_m) = _plan_block(lam_blocks[b], Pm, Dm, theta, N, B, C, coeffs, prices,
                                       pricing == PRICING_SEPARATE, nchunks=nchunks, **sli)
        M[b] = Mb
        xs[b] = plan.x; nx[b] = N * plan.x; nq[b] = N * plan.qp; ps[b] = p_solo
        wso[b] = w_s; wmi[b] = w_m
        values.append(plan.value)
        plans.append(dict(x=plan.x.tolist(), ym=plan.ym.tolist(), ys=plan.ys.tolist(), qp=plan.qp.tolist(),
                          qd=plan.qd.tolist()))
    if qcap is None:
        qcap = max(256, _next_pow2(4.0 * float(nq.max()) + 64.0 * math.sqrt(N)))
    fixed = lengths is None
    inp = SimInputs(
        name=name, I=I, N=N, R=R, B=B, C=C, nblk=nblk, gate=gate, router=router, placement=placement,
        pricing=pricing, length_mode=LENGTH_FIXED if fixed else LENGTH_TABLE, qcap=int(qcap), hist=hist,
        seed=seed, block_len=float(block_len),
        P=np.asarray(P_fixed if fixed else np.rint(Pm), np.uint32),
        D=np.asarray(D_fixed if fixed else np.rint(Dm), np.uint32),
        theta=theta.copy(), prio_rank=lp.priority_ranks(Pm, Dm),
        rates=np.ascontiguousarray(lam_blocks), lengths=lengths,
        prices=np.asarray(prices, float), coeffs=np.asarray(coeffs, float).copy(),
        M=M, xstar=xs, n_xstar=nx, n_qpstar=nq, p_solo=ps, w_solo=wso, w_mix=wmi,
        meta=dict(lp_value=values, plan=plans, Pm=list(map(float, Pm)), Dm=list(map(float, Dm)),
                  horizon_iters=int(horizon_iters), tau_ref=tau_ref(coeffs, B)),
    )
    inp.validate()
    return inp


def _capacity(pi, Pm, Dm, B, C, coeffs, nchunks=None):
    return _capacity_cached(tuple(map(float, pi)), tuple(map(float, Pm)), tuple(map(float, Dm)), int(B), int(C),
                            tuple(map(float, coeffs)), None if nchunks is None else tuple(map(float, nchunks)))


@functools.lru_cache(maxsize=None)
def _capacity_cached(pi, Pm, Dm, B, C, coeffs, nchunks):
    """Fluid capacity: the largest total per-GPU rate s with lambda = s*pi servable without queues, the
    iteration times being those of the batches that this load itself induces (bisection on s)."""
    pi = np.asarray(pi, float)
    coeffs = np.asarray(coeffs, float)
    w = np.asarray(Pm, float) + np.asarray(Dm, float)      # any positive weights: the question is feasibility
    ck = dict(beta=float(coeffs[1]), nchunks=np.asarray(nchunks, float)) if nchunks is not None else {}

    def served_all(s):
        lam = s * pi
        def solve(tm, ts):
            return lp.solve_plan(lam, Pm, Dm, np.zeros(len(pi)), B, C, tm, ts, 1.0, 1.0, **ck)
        _, _, plan = lp.consistent_taus(coeffs, B, C, solve)
        return plan.value >= float(np.dot(lam, w)) * (1.0 - 1e-7)

    tm, ts = lp.nominal_taus(coeffs, B, C)
    lo = lp.fluid_capacity(pi, Pm, Dm, B, C, tm, ts, **ck)  # full batches are the slowest: a safe lower bound
    if coeffs[2] == 0.0 and coeffs[4] == 0.0:
        return lo
    hi = lo
    while served_all(hi):
        lo, hi = hi, hi * 1.5
    for _ in range(40):
        mid = 0.5 * (lo + hi)
        if served_all(mid):
            lo = mid
        else:
            hi = mid
    return lo


def cfg0(placement=PLACE_LEAST_LOADED, R=16, horizon_iters=10_000) -> SimInputs:
    """Tiny instance: 2 fixed-length classes, N=4, B=32, 0.9 of fluid capacity, bundled (1, 2)."""
    P = [256, 1024]; D = [64, 256]; pi = np.array([0.5, 0.5])
    s = _capacity(pi, P, D, 32, 256, COEFFS_BENCH)
    inp = build("cfg0", N=4, R=R, B=32, C=256, Pm=P, Dm=D, lam_blocks=0.9 * s * pi, theta=[0.0, 0.0],
                prices=[1.0, 2.0], coeffs=COEFFS_BENCH, gate=GATE_OCCUPANCY, router=ROUTER_SOLO_FIRST,
                placement=placement, pricing=PRICING_BUNDLED, P_fixed=P, D_fixed=D, seed=0, qcap=4096,
                horizon_iters=horizon_iters)
    inp.meta["capacity"] = s
    return inp


_LN2CLASS = (((5.0, 0.5), (6.0, 0.5)), ((7.5, 0.6), (4.0, 0.5)))


def cfg1(placement=PLACE_LEAST_LOADED, R=1024, horizon_iters=100_000) -> SimInputs:
    """Two lognormal classes, N=64, B=128, separate pricing (0.5, 1.5), 0.9 of fluid capacity."""
    tabs = _two_class_tables()
    Pm = [table_mean(tabs[i, 0]) for i in range(2)]
    Dm = [table_mean(tabs[i, 1]) for i in range(2)]
    nch = [table_mean_chunks(tabs[i, 0], 256) for i in range(2)]
    pi = np.array([0.5, 0.5])
    s = _capacity(pi, Pm, Dm, 128, 256, COEFFS_BENCH, nch)
    inp = build("cfg1", N=64, R=R, B=128, C=256, Pm=Pm, Dm=Dm, nchunks=nch, lam_blocks=0.9 * s * pi, theta=[0.0, 0.0],
                prices=[0.5, 1.5], coeffs=COEFFS_BENCH, gate=GATE_PRIORITY, router=ROUTER_SOLO_FIRST,
                placement=placement, pricing=PRICING_SEPARATE, lengths=tabs, seed=1, qcap=4096,
                horizon_iters=horizon_iters)
    inp.meta["capacity"] = s
    return inp


_IN_MED = (128, 512, 2048, 4096)
_OUT_MED = (512, 256, 128, 32)
_MIX4 = np.array([0.4, 0.3, 0.2, 0.1])


@functools.lru_cache(maxsize=None)
def _two_class_tables():
    tabs = lognormal_tables(_LN2CLASS)
    tabs.setflags(write=False)
    return tabs


@functools.lru_cache(maxsize=None)
def _four_class():
    tabs = lognormal_tables([((math.log(a), 0.7), (math.log(b), 0.7)) for a, b in zip(_IN_MED, _OUT_MED)])
    Pm = [table_mean(tabs[i, 0]) for i in range(4)]
    Dm = [table_mean(tabs[i, 1]) for i in range(4)]
    nch = [table_mean_chunks(tabs[i, 0], 256) for i in range(4)]
    tabs.setflags(write=False)
    return tabs, Pm, Dm, nch


def cfg2(N=512, placement=PLACE_LEAST_LOADED, R=4096, horizon_iters=100_000) -> SimInputs:
    """Four lognormal classes at 1.05 of fluid capacity (patience 0.1/s so the excess leaves), bundled."""
    tabs, Pm, Dm, nch = _four_class()
    s = _capacity(_MIX4, Pm, Dm, 256, 256, COEFFS_BENCH, nch)
    inp = build("cfg2", N=N, R=R, B=256, C=256, Pm=Pm, Dm=Dm, nchunks=nch, lam_blocks=1.05 * s * _MIX4,
                theta=[0.1] * 4, prices=[1.0, 2.0], coeffs=COEFFS_BENCH, gate=GATE_OCCUPANCY,
                router=ROUTER_SOLO_FIRST, placement=placement, pricing=PRICING_BUNDLED, lengths=tabs,
                seed=2, horizon_iters=horizon_iters)
    inp.meta["capacity"] = s
    return inp


def cfg3(N=1024, placement=PLACE_LEAST_LOADED, R=2048, block_len=3600.0, nblk=24) -> SimInputs:
    """Time-varying demand: 24 blocks, sinusoid of amplitude 0.5 around 0.95 of capacity, per-block LP tables."""
    tabs, Pm, Dm, nch = _four_class()
    s = _capacity(_MIX4, Pm, Dm, 256, 256, COEFFS_BENCH, nch)
    lam = np.array([s * _MIX4 * (0.95 + 0.5 * math.sin(2.0 * math.pi * b / 24.0)) for b in range(nblk)])
    inp = build("cfg3", N=N, R=R, B=256, C=256, Pm=Pm, Dm=Dm, nchunks=nch, lam_blocks=lam, theta=[0.1] * 4,
                prices=[0.5, 1.5], coeffs=COEFFS_BENCH, gate=GATE_PRIORITY, router=ROUTER_SOLO_FIRST,
                placement=placement, pricing=PRICING_SEPARATE, lengths=tabs, seed=3, hist=1,
                block_len=block_len)
    inp.meta["capacity"] = s
    inp.meta["horizon_iters"] = int(math.ceil(nblk * block_len / tau_ref(COEFFS_BENCH, 256)))
    return inp


def cfg4(N=1024, placement=PLACE_LEAST_LOADED, R=8192, horizon_iters=100_000) -> SimInputs:
    """cfg2 workload under constrained-LP targets with the SLI-aware randomized router."""
    tabs, Pm, Dm, nch = _four_class()
    s = _capacity(_MIX4, Pm, Dm, 256, 256, COEFFS_BENCH, nch)
    inp = build(f"cfg4_N{N}", N=N, R=R, B=256, C=256, Pm=Pm, Dm=Dm, nchunks=nch, lam_blocks=1.05 * s * _MIX4,
                theta=[0.1] * 4, prices=[1.0, 2.0], coeffs=COEFFS_BENCH, gate=GATE_OCCUPANCY,
                router=ROUTER_SLI, placement=placement, pricing=PRICING_BUNDLED, lengths=tabs, seed=4,
                hist=1, sli=dict(qd_zero=True, min_admit_ratio=0.8, max_prefill_wait=2.0),
                horizon_iters=horizon_iters)
    inp.meta["capacity"] = s
    return inp


def paper_instance(n=50, R=5, router=ROUTER_SOLO_FIRST, gate=GATE_OCCUPANCY, placement=PLACE_RANDOM,
                   B=16, seed=100, horizon_iters=20_000, coeffs=COEFFS_PAPER) -> SimInputs:
    """P=(300,3000), D=(1000,400), lambda=(0.5,0.5), theta=(0.1,0.1), separate pricing (0.1, 0.2).

    The paper does not state B or the solo iteration time for this experiment; B=16 (the only
    batch cap it quotes) and 0.022 s are used.
    """
    P = [300, 3000]; D = [1000, 400]
    sli = dict(qd_zero=True) if router == ROUTER_SLI else None
    inp = build(f"paper_n{n}", N=n, R=R, B=B, C=256, Pm=P, Dm=D, lam_blocks=[0.5, 0.5], theta=[0.1, 0.1],
                prices=[0.1, 0.2], coeffs=coeffs, gate=gate, router=router, placement=placement,
                pricing=PRICING_SEPARATE, P_fixed=P, D_fixed=D, seed=seed, sli=sli,
                horizon_iters=horizon_iters)
    return inp


ABLATIONS = {   # label -> (gate, router, static planning)   [EC, additional ablation studies]
    "GG-SP": (GATE_OCCUPANCY, ROUTER_SOLO_FIRST, True),     # the full policy
    "FG-SP": (GATE_FCFS, ROUTER_SOLO_FIRST, True),          # FCFS admission, solo-first routing, static partition
    "GF-WSP": (GATE_OCCUPANCY, ROUTER_SOLO_FIRST, False),   # occupancy gate, one FCFS buffer served by whichever GPU has a slot: no solo group to prefer
    "GI-WSP": (GATE_OCCUPANCY, ROUTER_IMMEDIATE, False),    # occupancy gate, decode where the prefill ran, no partition
    "FI-WSP": (GATE_FCFS, ROUTER_IMMEDIATE, False),         # none of the three components
}


def ablation(policy="GG-SP", n=50, R=4, placement=PLACE_RANDOM, seed=100, horizon_iters=20_000, **kw) -> SimInputs:
    """The paper's two-class synthetic instance under one of the ablation policies of the EC ablation study.
    Without static planning every GPU may prefill (M = n); the LP targets still parameterise the occupancy gate."""
    gate, router, planned = ABLATIONS[policy]
    inp = paper_instance(n=n, R=R, gate=gate, router=router, placement=placement, seed=seed, horizon_iters=horizon_iters, **kw)
    if not planned:
        inp.M[:] = n
    inp.name = f"{policy}_n{n}"
    return inp


def aligned_instance(n=50, R=4, router=ROUTER_SOLO_FIRST, placement=PLACE_RANDOM, seed=5,
                     horizon_iters=60_000) -> SimInputs:
    """The paper's two-class synthetic instance with prompt lengths moved to multiples of the chunk size
    (256, 3072), so that a prefill takes exactly P/C iterations and the LP's rates (Eq. (4)) are exact
    for an iteration-level simulator."""
    P = [256, 3072]; D = [1000, 400]
    sli = dict(qd_zero=True) if router == ROUTER_SLI else None
    return build(f"aligned_n{n}", N=n, R=R, B=16, C=256, Pm=P, Dm=D, lam_blocks=[0.5, 0.5], theta=[0.1, 0.1],
                 prices=[0.1, 0.2], coeffs=COEFFS_PAPER, gate=GATE_OCCUPANCY, router=router, placement=placement,
                 pricing=PRICING_SEPARATE, P_fixed=P, D_fixed=D, seed=seed, sli=sli, horizon_iters=horizon_iters)


def single_class(N=1, B=3, C=256, P=512, D=2, lam=1.0, R=1, seed=7, coeffs=COEFFS_BENCH,
                 prices=(1.0, 2.0), theta=0.0, M=None, inject=None, placement=PLACE_LEAST_LOADED) -> SimInputs:
    """One fixed-length class; used by closed-form and hand-trace checks."""
    inp = build("single", N=N, R=R, B=B, C=C, Pm=[P], Dm=[D], lam_blocks=[lam], theta=[theta],
                prices=list(prices), coeffs=coeffs, gate=GATE_OCCUPANCY, router=ROUTER_SOLO_FIRST,
                placement=placement, pricing=PRICING_BUNDLED, P_fixed=[P], D_fixed=[D], seed=seed, qcap=256)
    if M is not None:
        inp.M[:] = M
    if inject is not None:
        t = np.array([e[0] for e in inject], np.float64)
        job = np.array([[e[1], e[2], e[3]] for e in inject], np.uint32).reshape(-1, 3)
        inp = inp.with_(inject_t=t, inject_job=job)
    return inp


def crowded(kind="decode", N=4, R=1, placement=PLACE_RANDOM, seed=None, M=None, router=ROUTER_SOLO_FIRST) -> SimInputs:
    """Two fixed-length classes with short patience, half of the GPUs mixed.  kind "decode": decode slots are the scarce
    resource (requests wait in, and abandon, the decode buffer); kind "prefill": prefill slots are scarce (requests
    abandon the prefill queues).  Per-GPU rates are fixed, so the congestion is the same at every cluster size."""
    P, D, lam, B, sd = ([300, 700], [60, 30], [9.0, 6.0], 4, 5) if kind == "decode" else ([1500, 2500], [10, 6], [8.0, 5.0], 8, 6)
    inp = build(f"crowded_{kind}_N{N}", N=N, R=R, B=B, C=256, Pm=P, Dm=D, lam_blocks=[lam], theta=[0.6, 0.9],
                prices=[1.0, 2.0], coeffs=COEFFS_BENCH, gate=GATE_OCCUPANCY, router=router,
                placement=placement, pricing=PRICING_BUNDLED, P_fixed=P, D_fixed=D, seed=sd if seed is None else seed,
                qcap=max(1024, _next_pow2(2.0 * N)))
    inp.M[:] = N // 2 if M is None else M
    return inp


def trace_replay(n=10, R=2, T=90.0, seed=42, placement=PLACE_RANDOM, coeffs=COEFFS_PAPER_KV):
    """Matched synthetic stand-in for the paper's trace replay (Section 6.2; the Azure traces are not
    redistributable): two classes ("code": long prompts, short outputs; "conversation": the reverse) with
    lognormal request-level lengths and Poisson timestamps generated here on the host, 10 GPUs, B = 16, C = 256,
    the KV-slope iteration law of the trace simulator.  Returns (inputs, class mean lengths)."""
    rng = np.random.default_rng(seed)
    spec = [(2.4 * n, 7.3, 0.8, 3.3, 0.9), (1.8 * n, 6.6, 0.9, 5.3, 0.7)]   # rate/s, mu_P, s_P, mu_D, s_D (congested)
    ts, jobs = [], []
    for cls, (rate, mp, sp, md, sd) in enumerate(spec):
        t = 0.0
        while True:
            t += rng.exponential(1.0 / rate)
            if t >= T:
                break
            P = int(np.clip(np.rint(np.exp(mp + sp * rng.standard_normal())), 1, 8192))
            D = int(np.clip(np.rint(np.exp(md + sd * rng.standard_normal())), 1, 8192))
            ts.append(t); jobs.append((cls, P, D))
    order = np.argsort(ts, kind="stable")
    ts = np.array(ts)[order]
    jobs = np.array(jobs, np.uint32)[order]
    Pm = [float(jobs[jobs[:, 0] == c, 1].mean()) for c in range(2)]
    Dm = [float(jobs[jobs[:, 0] == c, 2].mean()) for c in range(2)]
    lam0 = [1e-6, 1e-6]       # cold start: the controller knows nothing yet (lambda_min)
    inp = build(f"trace_n{n}", N=n, R=R, B=16, C=256, Pm=Pm, Dm=Dm, lam_blocks=lam0, theta=[0.0, 0.0],
                prices=[0.1, 0.2], coeffs=coeffs, gate=GATE_OCCUPANCY, router=ROUTER_SOLO_FIRST, placement=placement,
                pricing=PRICING_BUNDLED, P_fixed=[int(round(v)) for v in Pm], D_fixed=[int(round(v)) for v in Dm],
                seed=seed, qcap=4096)
    inp = inp.with_(inject_t=np.ascontiguousarray(ts, np.float64), inject_job=np.ascontiguousarray(jobs, np.uint32))
    return inp, Pm, Dm


def ctmc_instance(n=50, R=8, router=ROUTER_SOLO_FIRST, gate=GATE_OCCUPANCY, B=16, C=256, seed=11,
                  P=(300, 3000), D=(1000, 400), lam=(0.5, 0.5), theta=(0.1, 0.1), prices=(0.1, 0.2),
                  separate=True, coeffs=COEFFS_PAPER) -> CtmcInputs:
    """The exponential-service model of Section 2.3 on the paper's two-class synthetic instance (EC,
    "Convergence Analysis"): rates from Eq. (4) with tau = tau_mix(C) and gamma = 1/tau_solo, targets
    from the steady-state LP, M = ceil(n sum x*).  B and tau_solo as in `paper_instance`."""
    P = np.asarray(P, float); D = np.asarray(D, float); lam = np.asarray(lam, float); theta = np.asarray(theta, float)
    tau_mix, tau_solo = lp.nominal_taus(coeffs, B, C)
    mu_p, mu_m, mu_s = lp.service_rates(P, D, C, tau_mix, tau_solo)
    sli = dict(qd_zero=True) if router == ROUTER_SLI else {}
    plan = lp.solve_plan(lam, P, D, theta, B, C, tau_mix, tau_solo, prices[0], prices[1], separate=separate, **sli)
    I = len(P)
    inp = CtmcInputs(
        name=f"ctmc_n{n}", I=I, N=n, M=int(plan.M(n)), B=B, R=R, gate=gate, router=router,
        qcap=max(256, _next_pow2(64.0 * math.sqrt(n))), seed=seed,
        lam=lam.copy(), theta=theta.copy(), mu_p=np.asarray(mu_p, float), mu_m=np.asarray(mu_m, float),
        mu_s=np.asarray(mu_s, float), P=P.copy(), D=D.copy(), prices=np.asarray(prices, float),
        prio_rank=lp.priority_ranks(P, D), xstar=np.asarray(plan.x, float), n_xstar=n * np.asarray(plan.x, float),
        n_qpstar=n * np.asarray(plan.qp, float), p_solo=np.asarray(plan.p_solo(mu_m, mu_s), float),
        meta=dict(lp_value=float(plan.value), separate=bool(separate), tau_mix=tau_mix, tau_solo=tau_solo,
                  plan=dict(x=plan.x.tolist(), ym=plan.ym.tolist(), ys=plan.ys.tolist(), qp=plan.qp.tolist(),
                            qd=plan.qd.tolist())))
    inp.validate()
    return inp
