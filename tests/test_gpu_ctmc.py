"""GPU parity of the exponential-service model (qsim_ctmc_* through the C ABI) against its CPU oracle: integer
counters and end state bit-exact, time integrals within 1e-9 relative (clocks are bit-identical by construction)."""
import numpy as np
import pytest

from qsim_inputs import presets
from qsim_inputs.spec import CTMC_AREAS, CTMC_COUNTERS, CTMC_STATE, GATE_PRIORITY, ROUTER_SLI, ROUTER_SOLO_FIRST

pytestmark = pytest.mark.gpu
RTOL = 1e-9


def compare(gpu, ref, what):
    for k in CTMC_COUNTERS + CTMC_STATE + ("events",):
        assert np.array_equal(gpu[k], ref[k]), f"{what}: {k} differs at {np.argwhere(gpu[k] != ref[k])[:4].tolist()}"
    for k in CTMC_AREAS + ("T_elapsed",):
        assert np.allclose(gpu[k], ref[k], rtol=RTOL, atol=1e-300), f"{what}: {k}"


def gpu_run(inp, times):
    from paper_2602_02987_b200 import QSimCTMC
    sim = QSimCTMC(inp, device="cuda:0")
    for T in times:
        sim.run_until(T)
    st = sim.stats()
    sim.close()
    return st


@pytest.mark.parametrize("router,gate,theta,lam", [
    (ROUTER_SOLO_FIRST, 0, (0.1, 0.1), (0.5, 0.5)),        # the paper's synthetic instance
    (ROUTER_SLI, 0, (0.1, 0.1), (0.5, 0.5)),               # randomized router, two decode buffers
    (ROUTER_SOLO_FIRST, GATE_PRIORITY, (0.0, 0.3), (0.8, 0.8)),   # overload: buffers fill, one patient class, drops at a full buffer
    (ROUTER_SLI, GATE_PRIORITY, (0.3, 0.3), (0.9, 0.7)),
])
def test_ctmc_parity_element_by_element(router, gate, theta, lam):
    from oracle import run_ctmc_oracle
    inp = presets.ctmc_instance(n=24, R=70, router=router, gate=gate, theta=theta, lam=lam)     # 70: two blocks, ragged tail
    ref = run_ctmc_oracle(inp, 120.0)
    compare(gpu_run(inp, [120.0]), ref, "one call")
    compare(gpu_run(inp, [7.5, 7.5, 60.0, 120.0]), ref, "resumed")
    assert ref["abandoned_d"].sum() > 0 or min(theta) == 0.0
    # revenue per GPU (qsim_ctmc_revenue, Eq. (21)-(23)) against the oracle side's own arithmetic on the oracle's counters
    from oracle import ctmc_revenue_rate
    assert np.allclose(gpu_run(inp, [120.0])["_revenue_rate"], ctmc_revenue_rate(inp, ref), rtol=1e-12, atol=0)


def test_ctmc_full_size_in_the_bench_launch_configuration():
    from oracle import run_ctmc_oracle
    inp = presets.ctmc_instance(n=1000, R=37888, router=ROUTER_SLI)       # what `bench.py --workload ctmc` times
    gpu = gpu_run(inp, [10.0, 20.0])
    # sampled replications against the oracle (the Philox counter holds the global replication index)
    for r in (0, 18945, 37887):
        ref = run_ctmc_oracle(inp.with_(rep_offset=r, R=1), 20.0)
        for k in CTMC_COUNTERS + CTMC_STATE + ("events",):
            assert np.array_equal(gpu[k][r:r + 1], ref[k]), (r, k)
        for k in CTMC_AREAS:
            assert np.allclose(gpu[k][r:r + 1], ref[k], rtol=RTOL, atol=1e-300), (r, k)
    # flow balance Eq. (15)-(20) on every replication
    g = lambda k: gpu[k].astype(np.int64)
    assert np.array_equal(g("Qp"), g("arrivals") - g("admitted") - g("abandoned_p"))
    assert np.array_equal(g("X"), g("admitted") - g("prefill_done"))
    assert np.array_equal(g("Qd"), g("prefill_done") - g("placed_mixed") - g("placed_solo") - g("abandoned_d") - g("overflow_d"))
    assert np.array_equal(g("Ym") + g("Ys"), g("placed_mixed") + g("placed_solo") - g("done_mixed") - g("done_solo"))


def test_ctmc_eight_classes_and_argument_errors():
    from oracle import run_ctmc_oracle
    from paper_2602_02987_b200 import QSimCTMC, QSimError
    rng = np.random.default_rng(5)
    P = tuple(int(v) for v in rng.integers(200, 3000, 8)); D = tuple(int(v) for v in rng.integers(200, 3000, 8))
    inp = presets.ctmc_instance(n=16, R=33, P=P, D=D, lam=(0.12,) * 8, theta=(0.1,) * 8, router=ROUTER_SLI)
    compare(gpu_run(inp, [60.0]), run_ctmc_oracle(inp, 60.0), "eight classes")
    with pytest.raises(QSimError):
        QSimCTMC(inp.with_(M=inp.N + 1))
    with pytest.raises(QSimError):
        QSimCTMC(inp.with_(gate=2))


def test_ctmc_degenerate_cases():
    from oracle import run_ctmc_oracle
    base = presets.ctmc_instance(n=6, R=3)
    cases = {
        "one replication": base.with_(R=1),
        "no mixed GPU: nothing is ever admitted": base.with_(M=0),
        "every GPU mixed: no solo slots": base.with_(M=base.N),
        "B = 1: mixed GPUs hold no decode": base.with_(B=1),
        "a class without arrivals": base.with_(lam=np.array([0.5, 0.0])),
        "no patience": base.with_(theta=np.zeros(2)),
        "buffer of one request": base.with_(qcap=1, lam=np.array([2.0, 2.0])),
    }
    for what, inp in cases.items():
        ref = run_ctmc_oracle(inp, 50.0)
        compare(gpu_run(inp, [50.0]), ref, what)
    st = gpu_run(cases["no mixed GPU: nothing is ever admitted"], [50.0])
    assert st["admitted"].sum() == 0 and st["arrivals"].sum() > 0
    assert gpu_run(cases["buffer of one request"], [50.0])["overflow_d"].sum() > 0
    # an end time of zero processes nothing
    z = gpu_run(base, [0.0])
    assert z["events"].sum() == 0 and z["T_elapsed"].max() == 0.0


@pytest.mark.parametrize("seed", range(12))
def test_ctmc_random_configuration(seed):
    # random rates, targets and capacities (not an LP plan): parity does not depend on the inputs making sense
    from oracle import run_ctmc_oracle
    from qsim_inputs.spec import CtmcInputs
    rng = np.random.default_rng(700 + seed)
    I = int(rng.integers(1, 9)); N = int(rng.integers(1, 40)); M = int(rng.integers(0, N + 1)); B = int(rng.integers(1, 20))
    inp = CtmcInputs(name=f"rnd{seed}", I=I, N=N, M=M, B=B, R=int(rng.choice([1, 31, 33, 65])), gate=int(rng.integers(0, 2)),
                     router=int(rng.integers(0, 2)), qcap=int(rng.choice([1, 3, 64])), seed=seed,
                     lam=rng.random(I) * 0.6, theta=rng.choice([0.0, 0.1, 1.0], I), mu_p=0.5 + rng.random(I) * 3,
                     mu_m=0.05 + rng.random(I), mu_s=0.1 + rng.random(I) * 2, P=np.full(I, 100.0), D=np.full(I, 50.0),
                     prices=np.array([1.0, 2.0]), prio_rank=rng.permutation(I).astype(np.uint32),
                     xstar=rng.choice([0.0, 0.05, 0.2], I), n_xstar=rng.random(I) * N * 0.2, n_qpstar=rng.random(I) * 3,
                     p_solo=rng.choice([0.0, 0.3, 1.0], I))
    inp.validate()
    ref = run_ctmc_oracle(inp, 40.0)
    compare(gpu_run(inp, [11.0, 40.0]), ref, inp.name)
