"""Parity of the one-thread-per-replication kernels with the CPU oracle: the same seeded inputs, integer statistics
bit-exact, fp64 statistics within 1e-9 relative, per-GPU end state identical.  The family is forced here (by default
it is chosen only for thousands of replications), over every feature it simulates: the three gates, the solo-first and
the SLI-aware router with least-loaded placement, abandonment from both queues, blocks with role changes, histograms,
table-driven lengths, ragged and degenerate sizes, resumed and budget-limited runs."""
import contextlib
import os
import threading

import numpy as np
import pytest

from qsim_inputs import presets
from qsim_inputs.spec import (GATE_FCFS, GATE_OCCUPANCY, GATE_PRIORITY, PLACE_LEAST_LOADED, PLACE_RANDOM, ROUTER_SLI,
                              ROUTER_SOLO_FIRST)

from parity import assert_parity

pytestmark = pytest.mark.gpu


@contextlib.contextmanager
def family(name):
    keep = os.environ.get("QSIM_FAMILY")
    os.environ["QSIM_FAMILY"] = name
    try:
        yield
    finally:
        if keep is None:
            del os.environ["QSIM_FAMILY"]
        else:
            os.environ["QSIM_FAMILY"] = keep


def lane_run(inp, horizon, chunks=None, budget=None, expect_lane=True):
    from paper_2602_02987_b200 import QSim
    with family("lane"):
        sim = QSim(inp)
    assert (sim.layout_info()["warps"] == 0) == expect_lane
    if budget:
        sim.set_event_budget(budget)
    for h in (chunks or [horizon]):
        sim.run(h)
    st = sim.stats()
    state = [sim.server_state(r) for r in range(min(inp.R, 4))]
    sim.close()
    return st, state


def oracle_run(inp, horizon):
    from oracle import OracleSim
    out = [None] * inp.R

    def one(r):
        o = OracleSim(inp.with_(R=1, rep_offset=inp.rep_offset + r))
        o.run(horizon)
        out[r] = (o.stats(), o.server_state(0))
        o.close()

    th = [threading.Thread(target=one, args=(r,)) for r in range(inp.R)]
    for t in th:
        t.start()
    for t in th:
        t.join()
    st = {k: np.concatenate([out[r][0][k] for r in range(inp.R)]) for k in out[0][0]}
    return st, [out[r][1] for r in range(min(inp.R, 4))]


def check(inp, horizon, **kw):
    ref, rstate = oracle_run(inp, horizon)
    got, gstate = lane_run(inp, horizon, **kw)
    assert_parity(got, ref, what=f"lane family, {inp.name} N={inp.N} B={inp.B}")
    for a, b in zip(gstate, rstate):
        for k in a:
            assert np.array_equal(a[k], b[k]), (inp.name, "GPU state", k)
    return ref


def test_cfg0_whole():
    st = check(presets.cfg0(), 10_000)
    assert st["overflow"].sum() == 0 and int(st["iters_mixed"].sum() + st["iters_solo"].sum()) > 400_000


@pytest.mark.parametrize("gate", [GATE_OCCUPANCY, GATE_PRIORITY, GATE_FCFS])
@pytest.mark.parametrize("router", [ROUTER_SOLO_FIRST, ROUTER_SLI])
def test_paper_instance_gates_and_routers(gate, router):
    # abandonment in both queues, decode backlog, 37 GPUs, 40 replications (more than one warp of lanes)
    st = check(presets.paper_instance(n=37, R=40, gate=gate, placement=PLACE_LEAST_LOADED, router=router), 5000)
    assert st["abandoned_p"].sum() > 0


def test_cfg1_lognormal_tables_priority_gate():
    check(presets.cfg1(R=33), 1500)


def test_cfg2_overload_with_abandonment():
    st = check(presets.cfg2(N=64, R=8), 3000)
    assert st["abandoned_p"].sum() > 0
    check(presets.cfg2(N=512, R=3), 500)


def test_cfg3_blocks_role_changes_and_histograms():
    inp = presets.cfg3(N=96, R=6, block_len=1.0)
    st = check(inp, inp.meta["horizon_iters"])
    assert st["hist_ttft"].sum() == st["prefill_done"].sum()
    assert st["hist_tpot"].sum() == (st["done_mixed"] + st["done_solo"]).sum()
    assert len(set(inp.M.tolist())) > 2


@pytest.mark.parametrize("N,H", [(16, 1500), (64, 900), (100, 600), (256, 500)])
def test_cfg4_sli_router_constrained_targets(N, H):
    check(presets.cfg4(N=N, R=4), H)


@pytest.mark.parametrize("kind,N,H", [("decode", 4, 20_000), ("decode", 530, 500), ("prefill", 4, 20_000), ("prefill", 300, 900)])
def test_crowded_queues_and_buffers(kind, N, H):
    st = check(presets.crowded(kind, N=N, R=3, placement=PLACE_LEAST_LOADED), H)
    assert (st["abandoned_d"] if kind == "decode" else st["abandoned_p"]).sum() > 500


def test_crowded_with_the_sli_router_two_buffers():
    st = check(presets.crowded("decode", N=40, R=5, placement=PLACE_LEAST_LOADED, router=ROUTER_SLI).with_(
        p_solo=np.array([[0.6, 0.3]])), 4000)
    assert st["abandoned_d"].sum() > 100 and st["placed_mixed"].sum() > 0 and st["placed_solo"].sum() > 0


@pytest.mark.parametrize("N,H", [(1024, 500), (4096, 300)])
def test_large_clusters(N, H):
    st = check(presets.cfg4(N=N, R=2), H)
    assert (st["done_mixed"] + st["done_solo"]).sum() > 1000


def test_degenerate_sizes():
    check(presets.single_class(N=2, B=1, P=300, D=3, lam=5.0, theta=0.5, R=3, M=1), 20_000)
    check(presets.single_class(N=1, B=4, P=8192, D=8192, lam=0.05, R=2, M=1), 40_000)
    check(presets.single_class(N=9, B=9, P=600, D=40, lam=4.0, theta=0.1, R=2, M=4), 5000)
    inp = presets.single_class(N=3, B=4, lam=1.0, R=2)
    st, _ = lane_run(inp.with_(rates=np.zeros((1, 1))), 1000)
    assert st["events"].sum() == 0 and st["T_elapsed"][0] > 0


def test_tiny_queue_capacity_overflows_identically():
    st = check(presets.cfg0(R=3, horizon_iters=3000).with_(qcap=2), 3000)
    assert st["overflow"].sum() > 0


def test_small_queue_with_abandonment_from_inside():
    # eight positions per class queue, short patience: requests leave from inside the ring, positions run out while
    # fewer than eight wait (the ring is packed again), and arrivals overflow when eight do wait
    inp = presets.crowded("prefill", N=4, R=6, placement=PLACE_LEAST_LOADED).with_(qcap=8)
    st = check(inp, 20_000)
    assert st["overflow"].sum() > 0 and st["abandoned_p"].sum() > 500


def test_resumed_and_budget_limited_runs_are_identical():
    inp = presets.cfg2(N=48, R=5)
    a, sa = lane_run(inp, 3000)
    b, sb = lane_run(inp, 3000, chunks=[700, 1300, 1000])
    c, sc = lane_run(inp, 3000, budget=5000)
    for k in a:       # one thread adds every sum in event order: pieces give the same bits
        assert np.array_equal(a[k], b[k]), ("chunks", k)
        assert np.array_equal(a[k], c[k]), ("budget", k)
    for x, y, z in zip(sa, sb, sc):
        for k in x:
            assert np.array_equal(x[k], y[k]) and np.array_equal(x[k], z[k])


def test_checkpoint_reset_and_replication_offset():
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    inp = presets.cfg4(N=40, R=4)
    with family("lane"):
        sim = QSim(inp)
        sim.run(400)
        saved = sim.checkpoint()
        sim.close()
        sim = QSim(inp, checkpoint=saved)
        sim.run(300); sim.reset_stats(); sim.run(500)
        got = sim.stats()
        sim.close()
        lo = QSim(inp.with_(R=3)); lo.run(1200); a = lo.stats(); lo.close()
        hi = QSim(inp.with_(R=1, rep_offset=3)); hi.run(1200); b = hi.stats(); hi.close()
        whole = QSim(inp); whole.run(1200); w = whole.stats(); whole.close()
    o = OracleSim(inp); o.run(700); o.reset_stats(); o.run(500)
    assert_parity(got, o.stats(), what="lane family: checkpoint, resume, reset")
    o.close()
    for k in w:
        assert np.array_equal(w[k], np.concatenate([a[k], b[k]])), k


def test_the_two_families_agree_and_unsupported_modes_fall_back():
    from paper_2602_02987_b200 import QSim
    inp = presets.cfg2(N=130, R=6)
    lane, _ = lane_run(inp, 800)
    with family("warp"):
        sim = QSim(inp); sim.run(800); warp = sim.stats(); sim.close()
    assert_parity(lane, warp, what="lane family against warp family")
    # random placement is simulated by the warp-per-replication kernels only
    check(presets.paper_instance(n=20, R=3, placement=PLACE_RANDOM), 2000, expect_lane=False)


def test_whole_runs_in_waves_do_not_depend_on_the_wave_size():
    """qsim_simulate_waves: replications simulated a wave at a time in one bounded workspace.  Random streams are keyed by
    the global replication index, so waves of 64, of 148 and one wave of all give identical statistics, equal to the
    resident run's, in both kernel families."""
    from paper_2602_02987_b200 import QSim, simulate_waves
    inp = presets.cfg4(N=48, R=300)
    H = 400
    resident = {}
    for fam in ("warp", "lane"):
        with family(fam):
            sim = QSim(inp); sim.run(H); whole = resident[fam] = sim.stats(); sim.close()
            a = simulate_waves(inp, H, wave=64)
            b = simulate_waves(inp, H, wave=148)
            c = simulate_waves(inp, H, wave=0)
        assert (a["_waves"], b["_waves"], c["_waves"]) == (5, 3, 1)
        for k in whole:
            if k.startswith("hist"):
                continue
            assert np.array_equal(a[k], whole[k]) and np.array_equal(b[k], whole[k]) and np.array_equal(c[k], whole[k]), (fam, k)
        for k in a["_totals"]:      # totals are added in replication order whatever the waves
            assert np.array_equal(a["_totals"][k], b["_totals"][k]) and np.array_equal(a["_totals"][k], c["_totals"][k]), (fam, k)
    # a shard of a larger job: the offset composes with the waves
    with family("warp"):
        tail = simulate_waves(inp.with_(R=100, rep_offset=200), H, wave=33)
    for k in resident["warp"]:
        if not k.startswith("hist"):
            assert np.array_equal(tail[k], resident["warp"][k][200:]), k
