"""Pins of two parts of the oracle that the other trajectory and replay tests do not reach: the KV-token bookkeeping
behind the KV slope of the iteration time (Section 6.1, solo fit T_solo(K)), and the change of a GPU's role when the
number of mixed GPUs changes at a block boundary (Section 6.2: nothing running is pre-empted, the new split governs
later placement and admission; caps of Eq. (12)-(14)).  Also: the choices the paper makes uniformly at random are
uniform, and deliberately broken copies of the oracle fail these pins."""
import contextlib
import os

import numpy as np
import pytest

import oracle.qsim_oracle as orc
from oracle import OracleSim
from qsim_inputs import presets
from qsim_inputs.spec import (GATE_OCCUPANCY, PLACE_LEAST_LOADED, PLACE_RANDOM, PRICING_BUNDLED, ROUTER_SOLO_FIRST)

from replay import Replay

GOLD = os.path.join(os.path.dirname(__file__), "golden")
JOB = {c: k for k, c in enumerate("abcdefghi")}


def _load(name):
    return [line.split() for line in open(os.path.join(GOLD, name)) if line.strip() and not line.startswith("#")]


def _run(inp, iters, cap=1 << 16):
    sim = OracleSim(inp, trace_cap=cap)
    sim.run(iters)
    assert not sim.trace_overflowed()
    tr, st = sim.trace(), sim.stats()
    sim.close()
    return tr, st


# ---------------------------------------------------------------------------------------------------
# KV slope
# ---------------------------------------------------------------------------------------------------
def kv_case():
    return presets.single_class(N=1, B=3, C=256, P=256, D=2, M=1, coeffs=presets.COEFFS_PAPER_KV,
                                inject=[(0.0, 0, 256, 2), (0.001, 0, 300, 2)])


def check_kv_trajectory():
    tr, st = _run(kv_case(), 20)
    got = [(e["t"], e["type"], e["job"]) for e in tr if e["type"] in ("ITER_END", "PREFILL_DONE", "DECODE_DONE")]
    gold = _load("hand_trace_kv_slope.txt")
    assert len(got) == len(gold)
    for (t, typ, job), row in zip(got, gold):
        assert typ == row[1]
        assert abs(t - float(row[0])) < 1e-12, (t, row)
        if row[2] != "-":
            assert job == JOB[row[2]]
    assert abs(st["sum_ttft"][0, 0] - (0.033272 + 0.085727404)) < 1e-12
    assert abs(st["sum_tpot"][0, 0] - (0.026727702 + 0.008932454)) < 1e-12


def test_kv_slope_trajectory_worked_by_hand():
    check_kv_trajectory()


def check_kv_replay():
    # every iteration time of a congested run re-derived from the replayed batches: tau = law(p, d) + kappa K with
    # K summed request by request from prompt lengths and emitted tokens
    inp = presets.paper_instance(n=5, R=2, horizon_iters=6000, coeffs=presets.COEFFS_PAPER_KV)
    tr, st = _run(inp, 6000, cap=2_000_000)
    for r in range(inp.R):
        rp = Replay(inp, tr, rep=r).run()
        assert rp.n_events == st["events"][r]
    assert (st["done_mixed"] + st["done_solo"]).sum() > 50       # requests left, so K went down as well as up


def test_kv_slope_iteration_times_replayed_request_by_request():
    check_kv_replay()


# ---------------------------------------------------------------------------------------------------
# role change at a block boundary
# ---------------------------------------------------------------------------------------------------
def block_switch_case():
    times = (0.0, 0.001, 0.02, 0.021, 0.045, 0.046, 0.052, 0.101, 0.102)
    inp = presets.build("switch", N=3, R=1, B=2, C=256, Pm=[256], Dm=[20], lam_blocks=[[1.0], [1.0], [1.0]], theta=[0.0],
                        prices=[1.0, 2.0], coeffs=presets.COEFFS_BENCH, gate=GATE_OCCUPANCY, router=ROUTER_SOLO_FIRST,
                        placement=PLACE_LEAST_LOADED, pricing=PRICING_BUNDLED, P_fixed=[256], D_fixed=[20], seed=3,
                        qcap=64, block_len=0.05)
    inp.M[:] = [2, 1, 3]
    return inp.with_(inject_t=np.array(times), inject_job=np.array([[0, 256, 20]] * len(times), np.uint32))


def check_block_switch_trajectory():
    tr, st = _run(block_switch_case(), 25)
    got = [(e["t"], e["type"], e["job"], e["server"]) for e in tr
           if e["type"] in ("ADMIT", "PREFILL_DONE", "PLACE", "DECODE_DONE")]
    gold = _load("hand_trace_block_switch.txt")
    assert len(got) == len(gold), (len(got), len(gold))
    for (t, typ, job, srv), row in zip(got, gold):
        assert (typ, job, srv) == (row[1], JOB[row[2]], int(row[3])), ((t, typ, job, srv), row)
        assert abs(t - float(row[0])) < 1e-12
    assert abs(st["sum_tpot"][0, 0] - (0.0050975 + 0.005556)) < 1e-12
    assert [e["t"] for e in tr if e["type"] == "BLOCK"] == [0.05, 0.1]


def test_block_switch_trajectory_worked_by_hand():
    check_block_switch_trajectory()


def switching_poisson_case(seed=0):
    # one class, Poisson arrivals at a load that keeps decode slots scarce, three blocks with M = 2, 1, 3 of N = 3
    inp = presets.build("switch_poisson", N=3, R=2, B=3, C=256, Pm=[300], Dm=[12], lam_blocks=[[14.0], [14.0], [14.0]],
                        theta=[0.2], prices=[1.0, 2.0], coeffs=presets.COEFFS_BENCH, gate=GATE_OCCUPANCY,
                        router=ROUTER_SOLO_FIRST, placement=PLACE_RANDOM, pricing=PRICING_BUNDLED, P_fixed=[300],
                        D_fixed=[12], seed=seed, qcap=256, block_len=4.0)
    inp.M[:] = [2, 1, 3]
    return inp


def check_block_switch_replay():
    inp = switching_poisson_case()
    H = int(3 * 4.0 / inp.meta["tau_ref"]) + 1
    tr, st = _run(inp, H, cap=2_000_000)
    for r in range(inp.R):
        rp = Replay(inp, tr, rep=r).run()        # caps, tiers and admissions checked at every decision with the block's M
        assert rp.blk == 2
        assert rp.n_events == st["events"][r]
        # the cases of interest did occur: every GPU was full at some time, and requests waited in the decode buffer
        assert max(rp.max_load_seen) == inp.B
    assert st["area_Qd"].sum() > 0


def test_block_switch_replayed_with_role_changes():
    check_block_switch_replay()


# ---------------------------------------------------------------------------------------------------
# uniform choices
# ---------------------------------------------------------------------------------------------------
def _chi2_uniform(ranks, rng, bins=10):
    """Randomised probability-integral transform: (rank + U) / size is uniform on (0,1) iff the rank is uniform on
    0..size-1; returns the chi-square statistic over `bins` equal cells and the sample size."""
    r = np.array([a for a, k in ranks if k > 1], float)
    k = np.array([k for a, k in ranks if k > 1], float)
    u = (r + rng.random(r.size)) / k
    obs = np.histogram(u, bins=bins, range=(0.0, 1.0))[0]
    exp = r.size / bins
    return float(((obs - exp) ** 2 / exp).sum()), r.size


def check_uniform_choices():
    # Section 4.1 places a request on a GPU chosen uniformly among those of the tier that have room; memoryless
    # patience (Section 2.3) makes every waiting request of a class equally likely to be the one that leaves
    rng = np.random.default_rng(12345)
    place, ab_p, ab_d = [], [], []
    cases = [(presets.paper_instance(n=8, R=1, horizon_iters=12_000, placement=PLACE_RANDOM, seed=100), 12_000),
             (presets.crowded("decode"), 20_000), (presets.crowded("prefill"), 20_000)]
    for inp, H in cases:
        tr, _ = _run(inp, H, cap=4_000_000)
        rp = Replay(inp, tr, rep=0).run()
        place += rp.place_ranks + rp.admit_ranks
        ab_p += rp.abandon_p_ranks
        ab_d += rp.abandon_d_ranks
    # chi-square with 9 degrees of freedom: 33.7 is the 99.99 % point
    for name, ranks, need in (("placement", place, 3000), ("prefill-queue abandonment", ab_p, 2000),
                              ("decode-buffer abandonment", ab_d, 800)):
        stat, n = _chi2_uniform(ranks, rng)
        assert n >= need, (name, n)
        assert stat < 33.7, (name, stat, n)


def test_random_placement_and_abandonment_victims_are_uniform():
    check_uniform_choices()


# ---------------------------------------------------------------------------------------------------
# planted mistakes: each broken copy of the oracle must fail the pin that covers the line
# ---------------------------------------------------------------------------------------------------
@contextlib.contextmanager
def mutated_oracle(tmp_path, old, new):
    src = open(orc._SRC).read()
    assert src.count(old) == 1, f"mutation site not found exactly once: {old!r}"
    c_file = tmp_path / "mutant.c"
    c_file.write_text(src.replace(old, new))
    so = orc.compile_oracle(str(c_file), str(tmp_path / "libmutant.so"))
    keep = orc._lib
    orc._lib = orc.load_oracle(so)
    try:
        yield
    finally:
        orc._lib = keep


MUTANTS = [
    ("a finished request gives back only its prompt's KV tokens",
     "v->K -= (uint64_t)q->j.P + q->j.D;", "v->K -= (uint64_t)q->j.P;", (check_kv_trajectory, check_kv_replay)),
    ("a placed request's prompt is not added to the KV tokens",
     "v->K_pend += j.P;", "v->K_pend += 0;", (check_kv_trajectory, check_kv_replay)),
    ("emitted tokens do not grow the KV cache",
     "v->K += v->n_act;", "v->K += 0;", (check_kv_trajectory, check_kv_replay)),
    ("a demoted GPU that still prefills gets the full decode cap",
     "return (g < M || R->srv[g].pf_present) ? s->cfg.B - 1 : s->cfg.B;", "return (g < M) ? s->cfg.B - 1 : s->cfg.B;",
     (check_block_switch_trajectory, check_block_switch_replay)),
    ("a promoted GPU above the mixed cap takes a prefill",
     "default:               return g < M && !v->pf_present && v->n_dec <= s->cfg.B - 1;",
     "default:               return g < M && !v->pf_present;", (check_block_switch_trajectory, check_block_switch_replay)),
    ("a demoted GPU keeps taking prefills",
     "default:               return g < M && !v->pf_present && v->n_dec <= s->cfg.B - 1;",
     "default:               return !v->pf_present && v->n_dec <= s->cfg.B - 1;",
     (check_block_switch_trajectory, check_block_switch_replay)),
    ("the abandoning request is always the oldest",
     "uint32_t rank = (uint32_t)(((uint64_t)w[2] * Q) >> 32);\n    trace(s, r, ORC_EV_ABANDON_P",
     "uint32_t rank = 0;\n    trace(s, r, ORC_EV_ABANDON_P", (check_uniform_choices,)),
    ("random placement always takes the first GPU of the tier",
     "idx = (uint32_t)(((uint64_t)w[0] * cnt) >> 32);", "idx = 0;", (check_uniform_choices,)),
]


@pytest.mark.parametrize("what,old,new,checks", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_fails_its_pin(tmp_path, what, old, new, checks):
    with mutated_oracle(tmp_path, old, new):
        failed = []
        for chk in checks:
            try:
                chk()
            except AssertionError:
                failed.append(chk.__name__)
        assert failed, f"no pin noticed: {what}"
