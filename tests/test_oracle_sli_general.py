"""Pins for the general SLI-aware router (EC, "General SLI-aware Extension"): inside each pool the class that
gets a freed slot is drawn with probabilities proportional to varpi over the classes that wait, and the oldest
request of that class goes."""
import math

import numpy as np
import pytest

from oracle import OracleSim, run_oracle
from qsim_inputs import presets
from qsim_inputs.spec import ROUTER_SLI, ROUTER_SLI_GENERAL


def backlog_instance(w_solo, w_mix, **kw):
    # the paper's two-class instance: the decode stage is the bottleneck, so both buffers stay backlogged
    inp = presets.paper_instance(n=20, R=2, router=ROUTER_SLI_GENERAL, **kw)
    return inp.with_(p_solo=np.array([[0.8, 0.8]]), w_solo=np.array([w_solo], float), w_mix=np.array([w_mix], float))


def walk(inp, trace, rep):
    """Rebuilds both pool buffers from the trace; returns the selections made while both classes waited."""
    M = int(inp.M[0])
    buf = [[], []]                     # pool -> list of (cls, job) in arrival order
    picks = [[], []]                   # pool -> class chosen while >1 class waited
    starved = [[], []]                 # pool -> (chosen class, set of waiting classes)
    for e in (e for e in trace if e["rep"] == rep):
        typ, cls, g, job = e["type"], e["cls"], e["server"], e["job"]
        if typ == "PREFILL_DONE":
            buf[int(e["aux"])].append((cls, job))
        elif typ in ("ABANDON_D", "OVERFLOW") and (typ == "ABANDON_D" or g >= 0):
            pool = 0 if (cls, job) in buf[0] else 1
            buf[pool].remove((cls, job))
        elif typ == "PLACE":
            pool = 0 if g >= M else 1
            b = buf[pool]
            assert (cls, job) in b, "placed from the wrong pool"
            assert next(x for x in b if x[0] == cls) == (cls, job), "not FCFS within the class"
            waiting = {c for c, _ in b}
            if len(waiting) > 1:
                picks[pool].append(cls)
            starved[pool].append((cls, waiting))
            b.remove((cls, job))
    return picks, starved


def test_class_shares_follow_the_weights_under_backlog():
    inp = backlog_instance([0.25, 0.75], [0.6, 0.4])
    sim = OracleSim(inp, trace_cap=2_000_000)
    sim.run(12000)
    assert not sim.trace_overflowed()
    tr = sim.trace()
    for pool, w in ((0, 0.75), (1, 0.4)):
        chosen = []
        for r in range(inp.R):
            chosen += walk(inp, tr, r)[0][pool]
        n = len(chosen)
        assert n > 300, n
        share = sum(1 for c in chosen if c == 1) / n
        assert abs(share - w) < 4.0 * math.sqrt(w * (1 - w) / n), (pool, share, w, n)
    sim.close()


def test_zero_weight_class_waits_for_the_other():
    inp = backlog_instance([1.0, 0.0], [0.0, 1.0])
    sim = OracleSim(inp, trace_cap=2_000_000)
    sim.run(6000)
    tr = sim.trace()
    seen = 0
    for r in range(inp.R):
        _, starved = walk(inp, tr, r)
        for pool, loser in ((0, 1), (1, 0)):
            for cls, waiting in starved[pool]:
                if len(waiting) > 1:
                    assert cls != loser
                    seen += 1
    assert seen > 100
    sim.close()


def test_reduces_to_the_fcfs_pools_without_weights_or_with_one_class():
    # all weights zero: the head of the pool goes, which is the randomized router of Section 5.2
    a = run_oracle(backlog_instance([0.0, 0.0], [0.0, 0.0]), 4000)
    b = run_oracle(backlog_instance([0.3, 0.7], [0.3, 0.7]).with_(router=ROUTER_SLI), 4000)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    # one class: nothing to select
    one = presets.single_class(N=8, B=4, P=256, D=64, lam=3.0, R=2, M=4)
    one = one.with_(p_solo=np.array([[0.5]]), w_solo=np.array([[1.0]]), w_mix=np.array([[1.0]]))
    a = run_oracle(one.with_(router=ROUTER_SLI_GENERAL), 3000)
    b = run_oracle(one.with_(router=ROUTER_SLI), 3000)
    assert a["placed_solo"].sum() > 0 and a["placed_mixed"].sum() > 0
    for k in a:
        assert np.array_equal(a[k], b[k]), k


def test_weights_change_the_outcome_and_flow_balances():
    a = run_oracle(backlog_instance([0.25, 0.75], [0.5, 0.5]), 4000)
    b = run_oracle(backlog_instance([0.75, 0.25], [0.5, 0.5]), 4000)
    assert not np.array_equal(a["placed_solo"], b["placed_solo"])
    for st in (a, b):
        placed = st["placed_solo"] + st["placed_mixed"]
        assert np.array_equal(st["prefill_done"], placed + st["abandoned_d"] + st["overflow_d"] + st["Qd"])


def test_lp_weights_are_the_service_rate_shares():
    inp = presets.paper_instance(n=20, R=1, router=ROUTER_SLI_GENERAL)
    plan = inp.meta["plan"][0]
    for w, y in ((inp.w_solo[0], np.asarray(plan["ys"])), (inp.w_mix[0], np.asarray(plan["ym"]))):
        assert abs(w.sum() - 1.0) < 1e-12 or w.sum() == 0.0
        # equal decode lengths per class would give weights proportional to y*/D
        mu_ratio = (w[0] / w[1]) / (y[0] / y[1]) if (w[1] > 0 and y[1] > 0) else None
        if mu_ratio is not None:
            assert abs(mu_ratio - float(inp.D[1]) / float(inp.D[0])) < 1e-9
