"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

from qsim_inputs import presets
from qsim_inputs.spec import (GATE_OCCUPANCY, GATE_PRIORITY, PLACE_LEAST_LOADED, PLACE_RANDOM, ROUTER_SLI,
                              ROUTER_SOLO_FIRST)

from parity import assert_parity

pytestmark = pytest.mark.gpu


def gpu_run(inp, horizon, chunks=None, budget=None):
    from paper_2602_02987_b200 import QSim
    sim = QSim(inp)
    if budget:
        sim.set_event_budget(budget)
    for h in (chunks or [horizon]):
        sim.run(h)
    st = sim.stats()
    state = [sim.server_state(r) for r in range(min(inp.R, 2))]
    sim.close()
    return st, state


def oracle_run(inp, horizon, reps=None):
    from oracle import OracleSim
    sim = OracleSim(inp)
    if reps is None:
        sim.run(horizon)
    else:
        for r in reps:
            sim.run(horizon, r, r + 1)
    st = sim.stats()
    state = [sim.server_state(r) for r in range(min(inp.R, 2))]
    sim.close()
    return st, state


def check(inp, horizon, reps=None, **kw):
    g, gs = gpu_run(inp, horizon, **kw)
    o, os_ = oracle_run(inp, horizon, reps)
    assert_parity(g, o, rows=reps, what=inp.name)
    if reps is None:
        for a, b in zip(gs, os_):
            for k in a:
                assert np.array_equal(a[k], b[k]), (inp.name, "server state", k)
    return g


def test_cfg0_whole_both_placements():
    for placement in (PLACE_LEAST_LOADED, PLACE_RANDOM):
        inp = presets.cfg0(placement=placement)
        st = check(inp, 10_000)
        assert st["overflow"].sum() == 0
        assert int(st["iters_mixed"].sum() + st["iters_solo"].sum()) > 400_000


@pytest.mark.parametrize("gate", [GATE_OCCUPANCY, GATE_PRIORITY])
@pytest.mark.parametrize("placement", [PLACE_RANDOM, PLACE_LEAST_LOADED])
@pytest.mark.parametrize("router", [ROUTER_SOLO_FIRST, ROUTER_SLI])
def test_paper_instance_all_policy_modes(gate, placement, router):
    # abandonment in both queues, decode backlog, N not a multiple of 32
    inp = presets.paper_instance(n=37, R=6, gate=gate, placement=placement, router=router)
    check(inp, 6000)


def test_fcfs_gate_ablation():
    from qsim_inputs.spec import GATE_FCFS
    check(presets.paper_instance(n=20, R=4, gate=GATE_FCFS), 6000)
    check(presets.cfg1(R=4).with_(gate=GATE_FCFS), 1000)


@pytest.mark.parametrize("policy", ["GI-WSP", "FI-WSP"])
def test_immediate_decode_ablations(policy):
    # no router and no static partition (EC ablation study): a request decodes on the GPU that prefilled it
    for n, R, H, placement in ((12, 4, 3000, PLACE_RANDOM), (40, 3, 2500, PLACE_LEAST_LOADED), (600, 1, 150, PLACE_LEAST_LOADED)):
        inp = presets.ablation(policy, n=n, R=R, horizon_iters=H, placement=placement)
        st = check(inp, H)
        assert st["placed_solo"].sum() == 0 and st["Qd"].sum() == 0       # every GPU is mixed, nothing waits for a slot
        assert np.array_equal(st["placed_mixed"], st["prefill_done"])


def test_gate_and_fcfs_ablation_without_partition():
    # GF-WSP: every GPU is mixed, so the single FCFS buffer is served by whichever GPU has a slot
    for n, R, H in ((12, 4, 3000), (40, 3, 2500)):
        st = check(presets.ablation("GF-WSP", n=n, R=R, horizon_iters=H), H)
        assert st["placed_solo"].sum() == 0 and st["placed_mixed"].sum() > 0


@pytest.mark.parametrize("placement", [PLACE_RANDOM, PLACE_LEAST_LOADED])
def test_general_sli_router_class_selection(placement):
    # both pools backlogged with two classes: selections are drawn, requests leave from inside the buffers;
    # run in three pieces so that the selection ordinals cross launches
    from qsim_inputs.spec import ROUTER_SLI_GENERAL
    inp = presets.paper_instance(n=20, R=5, router=ROUTER_SLI_GENERAL, placement=placement)
    inp = inp.with_(p_solo=np.array([[0.8, 0.8]]), w_solo=np.array([[0.25, 0.75]]), w_mix=np.array([[0.6, 0.4]]))
    st = check(inp, 8000, chunks=[3000, 1, 4999])
    assert st["abandoned_d"].sum() > 0 and st["Qd"].sum() > 0
    # a cluster wide enough for the multi-warp instance, LP weights, one zero weight
    inp = presets.paper_instance(n=700, R=2, router=ROUTER_SLI_GENERAL, placement=placement)
    check(inp, 300)


def test_cfg1_subset_lognormal_tables_priority_gate():
    inp = presets.cfg1(R=8)
    check(inp, 1500)


def test_cfg2_subset_overload_with_abandonment():
    check(presets.cfg2(N=512, R=3), 400)
    st = check(presets.cfg2(N=64, R=4), 4000)
    assert st["abandoned_p"].sum() > 0


def test_cfg3_subset_block_tables_and_histograms():
    inp = presets.cfg3(N=96, R=4, block_len=1.0)
    H = inp.meta["horizon_iters"]
    st = check(inp, H)
    assert st["hist_ttft"].sum() == st["prefill_done"].sum()
    assert st["hist_tpot"].sum() == (st["done_mixed"] + st["done_solo"]).sum()


def test_latency_percentiles_from_the_histograms():
    from oracle import OracleSim, hist_percentiles
    from paper_2602_02987_b200 import QSim, QSimError
    inp = presets.cfg3(N=96, R=4, block_len=1.0)
    H = inp.meta["horizon_iters"]
    q = [0.5, 0.95, 0.99]
    sim = QSim(inp); sim.run(H)
    ttft, tpot = sim.latency_percentiles(q)
    sim.close()
    o = OracleSim(inp); o.run(H); st = o.stats(); o.close()
    assert np.array_equal(ttft, hist_percentiles(st["hist_ttft"], q))
    assert np.array_equal(tpot, hist_percentiles(st["hist_tpot"], q))
    assert (ttft[:, 0] <= ttft[:, 2]).all() and (tpot > 0).all()
    nohist = QSim(presets.cfg0(R=2)); nohist.run(100)
    with pytest.raises(QSimError):
        nohist.latency_percentiles(q)
    nohist.close()


def test_cfg4_subset_sli_router_constrained_targets():
    # N = 16: finish stamps on chip; N = 64, 128: global slot lists with 2 and 4 GPUs per lane; N = 256: run-time row count
    for N, H in ((16, 1200), (64, 800), (128, 500), (256, 500)):
        inp = presets.cfg4(N=N, R=3)
        check(inp, H)


def test_multi_warp_instances_large_clusters():
    # N >= 512 runs several warps per replication; each specialised instance and the generic one against the oracle
    import os
    inp = presets.cfg3(N=512, R=2, block_len=0.25)          # priority gate, blocks, histograms
    H = inp.meta["horizon_iters"]
    st = check(inp, H)
    assert st["hist_tpot"].sum() == (st["done_mixed"] + st["done_solo"]).sum()
    inp4 = presets.cfg4(N=512, R=2)                          # occupancy gate, SLI router, histograms
    g = check(inp4, 300)
    os.environ["QSIM_KERNEL"] = "generic"
    try:
        g2, _ = gpu_run(inp4, 300)
    finally:
        del os.environ["QSIM_KERNEL"]
    assert_parity(g2, g, what="generic multi-warp instance")


@pytest.mark.parametrize("preset,N,H", [("cfg4", 40, 900), ("cfg4", 100, 600), ("cfg4", 300, 300), ("cfg2", 33, 900),
                                         ("cfg2", 129, 500), ("cfg2", 520, 200)])
def test_ragged_cluster_sizes(preset, N, H):
    # cluster sizes that do not fill their last row of 32 GPUs, on every row-count variant of the specialised instances
    inp = getattr(presets, preset)(N=N, R=3)
    check(inp, H)


def test_large_n_one_replication():
    inp = presets.cfg4(N=4096, R=1)
    check(inp, 60)


def test_kv_slope_coefficients():
    inp = presets.paper_instance(n=12, R=4, coeffs=presets.COEFFS_PAPER_KV)
    check(inp, 20_000)


def test_resumable_and_event_budget_do_not_change_results():
    inp = presets.cfg2(N=48, R=4)
    a, _ = gpu_run(inp, 3000)
    b, _ = gpu_run(inp, 3000, chunks=[700, 1300, 1000])
    c, _ = gpu_run(inp, 3000, budget=5000)
    # integer statistics are identical; fp64 sums may be accumulated in another order when the look-ahead
    # windows are cut at different places
    for k in a:
        if a[k].dtype.kind == "f":
            assert np.allclose(a[k], b[k], rtol=1e-12, atol=0), ("chunks", k)
            assert np.allclose(a[k], c[k], rtol=1e-12, atol=0), ("budget", k)
        else:
            assert np.array_equal(a[k], b[k]), ("chunks", k)
            assert np.array_equal(a[k], c[k]), ("budget", k)


def test_checkpoint_and_resume_in_a_new_handle():
    from paper_2602_02987_b200 import QSim, QSimError
    for inp, h1, h2 in ((presets.cfg1(R=4), 700, 500), (presets.cfg4(N=512, R=2), 150, 150)):
        sim = QSim(inp)
        sim.run(h1)
        saved = sim.checkpoint()
        sim.close()
        sim = QSim(inp, checkpoint=saved)           # a new handle adopts the saved state and carries on
        sim.run(h2)
        got = sim.stats()
        sim.close()
        ref, _ = oracle_run(inp, h1 + h2)
        assert_parity(got, ref, what=f"{inp.name} resumed from a checkpoint")
    with pytest.raises(QSimError):
        QSim(presets.cfg1(R=5), checkpoint=saved)
    # same number of bytes, another seed: the workspace's fingerprint does not match the handle
    with pytest.raises(QSimError, match="configuration"):
        QSim(inp.with_(seed=inp.seed + 1), checkpoint=saved)


def test_replication_offset_shards_compose():
    inp = presets.cfg0(R=8, horizon_iters=2000)
    whole, _ = gpu_run(inp, 2000)
    lo, _ = gpu_run(inp.with_(R=5), 2000)
    hi, _ = gpu_run(inp.with_(R=3, rep_offset=5), 2000)
    for k in whole:
        assert np.array_equal(whole[k], np.concatenate([lo[k], hi[k]])), k


def test_reset_stats_and_host_entry_point():
    from paper_2602_02987_b200 import QSim, simulate_host
    inp = presets.cfg0(R=4, horizon_iters=3000)
    sim = QSim(inp)
    sim.run(1000); sim.reset_stats(); sim.run(2000)
    g = sim.stats(with_totals=True)
    sim.close()
    from oracle import OracleSim
    o = OracleSim(inp); o.run(1000); o.reset_stats(); o.run(2000)
    assert_parity(g, o.stats(), what="after reset")
    o.close()
    # totals are the sums over replications; revenue follows Eq. (22)
    assert int(g["_totals"]["arrivals"].sum()) == int(g["arrivals"].sum())
    T = g["T_elapsed"].sum()
    rev = (1.0 * g["tokens_in_completed"].sum() + 2.0 * g["tokens_out_completed"].sum()) / (inp.N * T)
    assert abs(g["_revenue_bundled"] - rev) <= 1e-12 * rev
    # the one-call host entry point gives the same statistics
    h = simulate_host(inp, 3000)
    ref, _ = gpu_run(inp, 3000)
    for k in ref:
        assert np.array_equal(ref[k], h[k]), k


def test_degenerate_sizes():
    # one GPU, one class, B = 1 (a mixed GPU then has no decode slot: jobs wait for the solo GPU)
    inp = presets.single_class(N=2, B=1, P=300, D=3, lam=5.0, theta=0.5, R=3, M=1)
    check(inp, 20_000)
    inp = presets.single_class(N=1, B=4, P=8192, D=8192, lam=0.05, R=2, M=1)
    check(inp, 40_000)
    # zero arrival rate: nothing ever happens
    inp = presets.single_class(N=3, B=4, lam=1.0, R=2)
    st, _ = gpu_run(inp.with_(rates=np.zeros((1, 1))), 1000)
    assert st["events"].sum() == 0 and st["T_elapsed"][0] > 0


def test_tiny_queue_capacity_overflows_identically():
    inp = presets.cfg0(R=3, horizon_iters=3000).with_(qcap=2)
    st = check(inp, 3000)
    assert st["overflow"].sum() > 0


def test_bad_arguments_are_rejected():
    from paper_2602_02987_b200 import QSim, QSimError
    good = presets.cfg0(R=2)
    for bad in (good.with_(N=5000), good.with_(qcap=0), good.with_(C=70000),
                good.with_(coeffs=np.array([0.0, 1e-5, 0, 0.005, 0, 0]))):
        with pytest.raises(QSimError):
            QSim(bad)


def test_cfg1_full_size_in_the_bench_launch_configuration():
    """The benchmark's own launch (R = 1024 replications, 10^5 iterations of horizon in one qsim_run): sampled
    replications against the oracle one by one, and the flow-balance identities (Eq. (15)-(20)) on all of them."""
    import threading
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    inp = presets.cfg1(R=1024)
    H = 100_000
    sim = QSim(inp)
    sim.run(H)
    g = sim.stats()
    sim.close()
    sample = [0, 517, 1023]
    ref = {}

    def one(r):
        o = OracleSim(inp.with_(R=1, rep_offset=r))
        o.run(H)
        ref[r] = o.stats()
        o.close()

    threads = [threading.Thread(target=one, args=(r,)) for r in sample]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    for r in sample:
        got = {k: v[r:r + 1] for k, v in g.items()}
        assert_parity(got, ref[r], what=f"cfg1 full size, replication {r}")
    u = {k: v.astype(np.int64) for k, v in g.items() if v.dtype.kind in "ui"}
    assert np.array_equal(u["Qp"], u["arrivals"] - u["admitted"] - u["abandoned_p"] - u["overflow"])
    assert np.array_equal(u["X"], u["admitted"] - u["prefill_done"])
    assert np.array_equal(u["Qd"], u["prefill_done"] - u["placed_mixed"] - u["placed_solo"] - u["abandoned_d"] - u["overflow_d"])
    assert np.array_equal(u["Ym"], u["placed_mixed"] - u["done_mixed"])
    assert np.array_equal(u["Ys"], u["placed_solo"] - u["done_solo"])
    assert u["overflow"].sum() == 0 and u["overflow_d"].sum() == 0
    its = (u["iters_mixed"] + u["iters_solo"])
    assert its.min() > 6_000_000
    # Poisson arrivals: counts across replications have mean n lambda T and dispersion 1
    T = g["T_elapsed"][0]
    for i in range(inp.I):
        mean = inp.N * inp.rates[0, i] * T
        a = g["arrivals"][:, i].astype(float)
        assert abs(a.mean() - mean) < 5.0 * np.sqrt(mean / a.size)
        assert abs(a.var(ddof=1) / mean - 1.0) < 5.0 * np.sqrt(2.0 / (a.size - 1))


def test_totals_reduced_on_the_device_are_the_host_totals_bit_for_bit():
    """qsim_stats with totals only sums on the device (integer counters exactly, fp64 statistics in replication order);
    the result must be the very bits of the host's sum over the per-replication records, in both kernel families."""
    import os
    from paper_2602_02987_b200 import QSim, simulate_host
    for fam, inp, H in (("warp", presets.cfg1(R=37), 600), ("lane", presets.cfg4(N=24, R=70), 700)):
        os.environ["QSIM_FAMILY"] = fam
        try:
            sim = QSim(inp)
            sim.run(H)
            full = sim.stats(with_totals=True)["_totals"]
            _, _, tot = sim.totals()
            sim.close()
        finally:
            del os.environ["QSIM_FAMILY"]
        for k, v in full.items():
            if v.ndim == 2:
                got = np.array([[getattr(tot.cls[i], k) for i in range(inp.I)]], v.dtype)
            else:
                got = np.array([getattr(tot, k)], v.dtype)
            assert np.array_equal(got, v), (fam, k, got, v)
    # the one-call host entry point with totals only
    inp = presets.cfg0(R=5, horizon_iters=1500)
    a = simulate_host(inp, 1500)["_totals"]
    b = simulate_host(inp, 1500, per_rep=False)["_totals"]
    for k in a:
        assert np.array_equal(a[k], b[k]), k
