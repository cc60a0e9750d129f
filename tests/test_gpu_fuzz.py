"""Seeded random configurations (sizes, class counts, gates, routers, placements, patience, pricing, histograms) on the
GPU against the oracle: integer statistics bit-exact, fp64 statistics within 1e-9, per-GPU end state identical."""
import numpy as np
import pytest

from qsim_inputs import presets
from qsim_inputs.spec import PRICING_BUNDLED, PRICING_SEPARATE

from parity import assert_parity

pytestmark = pytest.mark.gpu


def random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    I = int(rng.integers(1, 5))
    N = int(rng.choice([1, 2, 3, 7, 31, 32, 33, 45, 64, 65, 97, 130]))
    B = int(rng.choice([1, 2, 3, 16, 31, 32, 33, 64, 100]))
    C = int(rng.choice([64, 256, 1024]))
    P = [int(v) for v in rng.integers(20, 2500, I)]
    D = [int(v) for v in rng.integers(1, 400, I)]
    gate = int(rng.integers(0, 3))
    router = int(rng.choice([0, 1, 2, 3]))
    placement = int(rng.integers(0, 2))
    theta = [float(rng.choice([0.0, 0.05, 0.5])) for _ in range(I)]
    separate = bool(rng.integers(0, 2))
    coeffs = [presets.COEFFS_BENCH, presets.COEFFS_PAPER, presets.COEFFS_PAPER_KV][int(rng.integers(0, 3))]
    load = float(rng.choice([0.5, 0.9, 1.3]))
    pi = rng.dirichlet(np.ones(I))
    cap = presets._capacity(pi, P, D, max(B, 2), C, coeffs)
    lam = load * cap * pi
    inp = presets.build(f"fuzz{seed}", N=N, R=2, B=B, C=C, Pm=P, Dm=D, lam_blocks=lam, theta=theta,
                        prices=[0.3, 1.1], coeffs=coeffs, gate=gate, router=router, placement=placement,
                        pricing=PRICING_SEPARATE if separate else PRICING_BUNDLED, P_fixed=P, D_fixed=D,
                        seed=seed, hist=int(rng.integers(0, 2)), qcap=int(rng.choice([4, 64, 1024])))
    if router == 2:      # class-selection weights of the general SLI router
        inp = inp.with_(w_solo=rng.random((1, I)), w_mix=rng.random((1, I)))
    if router == 3 and rng.integers(0, 2):
        inp.M[:] = N     # no static partition
    return inp


@pytest.mark.parametrize("seed", range(24))
def test_random_configuration(seed):
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    inp = random_case(seed)
    H = int(np.random.default_rng(seed).choice([300, 1500, 4000]))
    sim = QSim(inp)
    for h in (H // 3, H - H // 3):
        sim.run(h)
    got = sim.stats()
    gstate = [sim.server_state(r) for r in range(inp.R)]
    sim.close()
    o = OracleSim(inp)
    o.run(H)
    ref = o.stats()
    ostate = [o.server_state(r) for r in range(inp.R)]
    o.close()
    assert_parity(got, ref, what=f"{inp.name}: N={inp.N} B={inp.B} I={inp.I} gate={inp.gate} router={inp.router} placement={inp.placement}")
    for a, b in zip(gstate, ostate):
        for k in a:
            assert np.array_equal(a[k], b[k]), (inp.name, "GPU state", k)


@pytest.mark.parametrize("seed", range(24))
def test_random_sizes_on_the_benchmark_feature_sets(seed):
    # the feature sets that have their own kernel instances (cfg1, cfg2, cfg4 recipes) on random cluster sizes and decode caps
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    rng = np.random.default_rng(5000 + seed)
    recipe = [presets.cfg1, presets.cfg2, presets.cfg4][seed % 3]
    N = int(rng.choice([1, 5, 32, 33, 64, 70, 128, 129, 200, 512, 530, 1024, 2049]))
    B = int(rng.choice([2, 17, 32, 100, 128, 256]))
    kw = {} if recipe is presets.cfg1 else {"N": N}
    inp = recipe(R=2, **kw)
    if recipe is presets.cfg1:
        N = int(rng.choice([1, 5, 33, 64, 100]))
        inp = inp.with_(N=N, M=np.array([max(1, N // 3)], np.uint32), n_xstar=inp.xstar * N, n_qpstar=inp.n_qpstar * N / 64)
    inp = inp.with_(B=B, seed=seed)
    H = max(int(60_000 / max(N, 20)), 150)
    sim = QSim(inp); sim.run(H); got = sim.stats(); gstate = [sim.server_state(r) for r in range(inp.R)]; sim.close()
    o = OracleSim(inp); o.run(H); ref = o.stats(); ostate = [o.server_state(r) for r in range(inp.R)]; o.close()
    assert_parity(got, ref, what=f"{inp.name}: N={inp.N} B={inp.B}")
    for a, b in zip(gstate, ostate):
        for k in a:
            assert np.array_equal(a[k], b[k]), (inp.name, "GPU state", k)


@pytest.mark.parametrize("recipe,N,B", [("cfg2", 1024, 100), ("cfg4", 2049, 17), ("cfg2", 2049, 33), ("cfg4", 1023, 256)])
def test_sizes_around_the_warp_count_thresholds(recipe, N, B):
    # 1024 GPUs = 32 rows (two warps per replication, 1023 still one), 2049 = 65 rows (four warps, last row holds one GPU)
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    inp = getattr(presets, recipe)(N=N, R=2).with_(B=B, seed=N + B)
    H = 150
    sim = QSim(inp); sim.run(H); got = sim.stats(); gstate = [sim.server_state(r) for r in range(inp.R)]; sim.close()
    o = OracleSim(inp); o.run(H); ref = o.stats(); ostate = [o.server_state(r) for r in range(inp.R)]; o.close()
    assert_parity(got, ref, what=f"{inp.name}: N={inp.N} B={inp.B}")
    for a, b in zip(gstate, ostate):
        for k in a:
            assert np.array_equal(a[k], b[k]), (inp.name, "GPU state", k)
