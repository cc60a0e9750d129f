"""Paper-stated invariants checked on oracle runs: flow balance, capacity, FCFS, token-level service,
the gate and router rules, a finite-horizon Little identity and resumability."""
import numpy as np
import pytest

from oracle import OracleSim, run_oracle
from qsim_inputs import presets
from qsim_inputs.spec import (GATE_FCFS, GATE_OCCUPANCY, GATE_PRIORITY, PLACE_LEAST_LOADED, PLACE_RANDOM, ROUTER_SLI)

from replay import Replay, expected_counts, isclose


def flow_balance(st):
    """Eq. (15)-(20) with zero initial state."""
    u = {k: st[k].astype(np.int64) for k in st if st[k].dtype.kind in "ui"}
    assert np.array_equal(u["Qp"], u["arrivals"] - u["admitted"] - u["abandoned_p"] - u["overflow"])      # (15)
    assert np.array_equal(u["X"], u["admitted"] - u["prefill_done"])                                        # (16)
    assert np.array_equal(u["Qd"], u["prefill_done"] - u["placed_mixed"] - u["placed_solo"]
                          - u["abandoned_d"] - u["overflow_d"])                                             # (17)
    assert np.array_equal(u["Ym"] + u["Ys"], u["placed_mixed"] + u["placed_solo"]
                          - u["done_mixed"] - u["done_solo"])                                               # (20)
    assert np.array_equal(u["Ym"], u["placed_mixed"] - u["done_mixed"])
    assert np.array_equal(u["Ys"], u["placed_solo"] - u["done_solo"])


def small_cases():
    yield presets.cfg0(R=2, horizon_iters=400)
    yield presets.cfg0(R=2, horizon_iters=400, placement=PLACE_RANDOM)
    yield presets.cfg0(R=1, horizon_iters=400).with_(gate=GATE_PRIORITY)
    yield presets.cfg0(R=1, horizon_iters=400).with_(gate=GATE_FCFS)
    yield presets.paper_instance(n=6, R=1, horizon_iters=1500, gate=GATE_FCFS)
    yield presets.paper_instance(n=5, R=2, horizon_iters=1500)
    yield presets.paper_instance(n=8, R=1, horizon_iters=1500, placement=PLACE_LEAST_LOADED, gate=GATE_PRIORITY)
    yield presets.ablation("GF-WSP", n=5, R=1, horizon_iters=1500)
    yield presets.ablation("GI-WSP", n=5, R=2, horizon_iters=1500)
    yield presets.ablation("FI-WSP", n=6, R=1, horizon_iters=1500, placement=PLACE_LEAST_LOADED)
    c1 = presets.cfg1(R=1, horizon_iters=150)
    yield c1.with_(N=6, M=np.array([4], np.uint32), n_xstar=c1.xstar * 6, rates=c1.rates * 1.2)


@pytest.mark.parametrize("inp", list(small_cases()), ids=lambda c: f"{c.name}-g{c.gate}-p{c.placement}-r{c.router}")
def test_replay_of_every_event(inp):
    sim = OracleSim(inp, trace_cap=2_000_000)
    H = inp.meta["horizon_iters"]
    sim.run(H)
    assert not sim.trace_overflowed()
    tr, st = sim.trace(), sim.stats()
    lengths = None
    if inp.length_mode == 1:
        # lengths are not in the trace: recover them from the decode/prefill behaviour is circular, so
        # only fixed-length cases get the token-level check; table cases check balance only
        flow_balance(st)
        return
    for r in range(inp.R):
        rp = Replay(inp, tr, rep=r).run(lengths)
        T = float(st["T_elapsed"][r])
        c = expected_counts(rp)
        for i in range(inp.I):
            assert c["arrivals"][i] == st["arrivals"][r, i]
            assert c["admitted"][i] == st["admitted"][r, i]
            assert c["prefill_done"][i] == st["prefill_done"][r, i]
            assert c["placed"][i] == st["placed_mixed"][r, i] + st["placed_solo"][r, i]
            assert c["done"][i] == st["done_mixed"][r, i] + st["done_solo"][r, i]
            assert c["abandoned_p"][i] == st["abandoned_p"][r, i]
            assert c["abandoned_d"][i] == st["abandoned_d"][r, i]
        # finite-horizon Little identity: integral of the count = sum over jobs of time in stage
        lit = rp.stage_time(T)
        for i in range(inp.I):
            assert isclose(lit["Qp"][i], st["area_Qp"][r, i])
            assert isclose(lit["X"][i], st["area_X"][r, i])
            assert isclose(lit["Qd"][i], st["area_Qd"][r, i])
            assert isclose(lit["Y"][i], st["area_Ym"][r, i] + st["area_Ys"][r, i])
        # latency sums re-derived job by job
        for i in range(inp.I):
            ttft = sum(j["t_pf"] - j["t_arr"] for (c_, _), j in rp.jobs.items() if c_ == i and "t_pf" in j)
            tpot = sum((j["t_done"] - j["t_pf"]) / j["D"] for (c_, _), j in rp.jobs.items()
                       if c_ == i and "t_done" in j)
            assert isclose(ttft, st["sum_ttft"][r, i]) and isclose(tpot, st["sum_tpot"][r, i])
        assert rp.n_events == st["events"][r]
    flow_balance(st)
    sim.close()


@pytest.mark.parametrize("make", [
    lambda: presets.cfg0(R=4, horizon_iters=3000),
    lambda: presets.cfg1(R=2, horizon_iters=300),
    lambda: presets.cfg2(N=16, R=2, horizon_iters=2000),
    lambda: presets.cfg3(N=16, R=2, block_len=2.0, nblk=6),
    lambda: presets.cfg4(N=16, R=2, horizon_iters=2000),
    lambda: presets.paper_instance(n=20, R=2, router=ROUTER_SLI, horizon_iters=3000),
], ids=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4", "paper-sli"])
def test_flow_balance_and_capacity_on_every_config(make):
    inp = make()
    sim = OracleSim(inp)
    sim.run(inp.meta["horizon_iters"])
    st = sim.stats()
    flow_balance(st)
    assert st["overflow"].sum() == 0 and st["overflow_d"].sum() == 0
    # Eq. (12)-(14) on the final state, per GPU
    for r in range(inp.R):
        s = sim.server_state(r)
        M = int(inp.M[-1])
        assert np.all(s["n_dec"] <= inp.B)
        assert np.all(s["pf_rem"][M:] == 0) or inp.nblk > 1
        assert np.all(s["n_dec"][s["pf_rem"] > 0] <= inp.B - 1)
        assert int((s["pf_rem"] > 0).sum()) == int(st["X"][r].sum())
        assert int(s["n_dec"].sum()) == int(st["Ym"][r].sum() + st["Ys"][r].sum())
    # tokens and completions agree with fixed lengths
    if inp.length_mode == 0:
        done = st["done_mixed"] + st["done_solo"]
        assert np.array_equal(st["tokens_out_completed"], done * inp.D.astype(np.uint64))
        assert np.array_equal(st["tokens_in_completed"], done * inp.P.astype(np.uint64))
        assert np.array_equal(st["tokens_in_prefilled"], st["prefill_done"] * inp.P.astype(np.uint64))
    sim.close()


def test_run_is_resumable_bit_for_bit():
    inp = presets.cfg2(N=8, R=2, horizon_iters=1500)
    a = OracleSim(inp); a.run(1500); sa = a.stats()
    b = OracleSim(inp); b.run(400); b.stats(); b.run(1100); sb = b.stats()
    for k in sa:
        assert np.array_equal(sa[k], sb[k]), k
    a.close(); b.close()


def test_replications_are_independent_streams_and_offsets_compose():
    inp = presets.cfg0(R=4, horizon_iters=800)
    whole = run_oracle(inp, 800)
    tail = run_oracle(inp.with_(R=2, rep_offset=2), 800)
    for k in whole:
        assert np.array_equal(whole[k][2:], tail[k]), k
    # different replications differ
    assert not np.array_equal(whole["arrivals"][0], whole["arrivals"][1])
    # arrivals do not depend on the policy (common random numbers)
    other = run_oracle(inp.with_(placement=PLACE_RANDOM, gate=GATE_PRIORITY), 800)
    assert np.array_equal(whole["arrivals"], other["arrivals"])


def test_reset_stats_discards_warm_up_but_keeps_state():
    inp = presets.cfg0(R=2, horizon_iters=2000)
    a = OracleSim(inp); a.run(500); s0 = a.stats(); a.reset_stats(); a.run(1500); s1 = a.stats()
    b = OracleSim(inp); b.run(2000); s2 = b.stats()
    for k in ("arrivals", "admitted", "done_mixed", "done_solo", "iters_mixed", "iters_solo", "events"):
        assert np.array_equal(s0[k] + s1[k], s2[k]), k
    for k in ("Qp", "X", "Qd", "Ym", "Ys"):
        assert np.array_equal(s1[k], s2[k])
    assert np.allclose(s0["area_X"] + s1["area_X"], s2["area_X"], rtol=1e-12)
    assert np.allclose(s0["T_elapsed"] + s1["T_elapsed"], s2["T_elapsed"], rtol=1e-15)
    a.close(); b.close()


def test_histogram_percentiles_bracket_the_exact_order_statistics():
    # TTFT / TPOT of every request re-derived from the event trace; the histogram percentile is the lower edge of the
    # bin that holds the ceil(q n)-th smallest latency
    from oracle import bin_lower_edge, hist_percentiles
    inp = presets.cfg0(R=2, horizon_iters=1500).with_(hist=1)
    sim = OracleSim(inp, trace_cap=2_000_000)
    sim.run(1500)
    tr, st = sim.trace(), sim.stats()
    q = [0.5, 0.9, 0.99, 1.0]
    pt, pp = hist_percentiles(st["hist_ttft"], q), hist_percentiles(st["hist_tpot"], q)
    jobs = {}
    for r in range(inp.R):
        rp = Replay(inp, tr, rep=r).run(None)
        for (c, j), rec in rp.jobs.items():
            jobs[(r, c, j)] = rec
    for i in range(inp.I):
        ttft = sorted(v["t_pf"] - v["t_arr"] for (r, c, j), v in jobs.items() if c == i and "t_pf" in v)
        tpot = sorted((v["t_done"] - v["t_pf"]) / v["D"] for (r, c, j), v in jobs.items() if c == i and "t_done" in v)
        assert len(ttft) == st["hist_ttft"][:, i].sum() and len(tpot) == st["hist_tpot"][:, i].sum()
        for k, qq in enumerate(q):
            for xs, p in ((ttft, pt[i, k]), (tpot, pp[i, k])):
                x = xs[int(np.ceil(qq * len(xs))) - 1]
                b = int(np.searchsorted(bin_lower_edge(np.arange(1024)), p, side="right")) - 1
                assert bin_lower_edge(np.array([b]))[0] == p
                assert p <= x < bin_lower_edge(np.array([b + 1]))[0] and x / p < 1.0 + 1.0 / 32 + 1e-12
