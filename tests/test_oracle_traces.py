"""Hand-worked trajectories (tests/golden) against the oracle's event trace."""
import os

import numpy as np
import pytest

from oracle import OracleSim
from qsim_inputs import presets

GOLD = os.path.join(os.path.dirname(__file__), "golden")
JOB = {"a": 0, "b": 1, "c": 2, "d": 3}


def _load(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        rows.append(line.split())
    return rows


def _trace(inp, iters):
    sim = OracleSim(inp, trace_cap=4096)
    sim.run(iters)
    tr, st = sim.trace(), sim.stats()
    state = sim.server_state(0)
    sim.close()
    return tr, st, state


def test_one_gpu_trajectory():
    inp = presets.single_class(N=1, B=3, C=256, P=512, D=2, M=1,
                               inject=[(0.0, 0, 512, 2), (0.001, 0, 512, 2)])
    tr, st, _ = _trace(inp, 20)
    got = [(e["t"], e["type"], e["job"]) for e in tr if e["type"] in ("ITER_END", "PREFILL_DONE", "DECODE_DONE")]
    gold = _load("hand_trace_1gpu.txt")
    assert len(got) == len(gold)
    for (t, typ, job), row in zip(got, gold):
        assert typ == row[1]
        assert abs(t - float(row[0])) < 1e-12
        if row[2] != "-":
            assert job == JOB[row[2]]
    assert abs(st["sum_ttft"][0, 0] - (0.02024 + 0.03958)) < 1e-12
    assert abs(st["sum_tpot"][0, 0] - (0.01017 + 0.00505)) < 1e-12
    assert int(st["iters_mixed"][0] + st["iters_solo"][0]) == 6
    c_p, c_d = inp.prices
    bundled = c_p * st["tokens_in_completed"].sum() + c_d * st["tokens_out_completed"].sum()
    separate = c_p * st["tokens_in_prefilled"].sum() + c_d * st["tokens_out_completed"].sum()
    assert bundled == separate == 1032.0


def test_two_gpu_trajectory_solo_first_then_mixed_then_buffer():
    inj = [(0.0, 0, 256, 6), (0.001, 0, 256, 6), (0.002, 0, 256, 6), (0.003, 0, 256, 6)]
    inp = presets.single_class(N=2, B=2, C=256, P=256, D=6, M=1, inject=inj)
    tr, st, _ = _trace(inp, 40)
    got = [(e["t"], e["type"], e["job"], e["server"]) for e in tr
           if e["type"] in ("PREFILL_DONE", "PLACE", "DECODE_DONE")]
    gold = _load("hand_trace_2gpu.txt")
    assert len(got) == len(gold)
    for (t, typ, job, srv), row in zip(got, gold):
        assert (typ, job, srv) == (row[1], JOB[row[2]], int(row[3]))
        assert abs(t - float(row[0])) < 1e-12
    ends = {0: [], 1: []}
    for e in tr:
        if e["type"] == "ITER_END":
            ends[e["server"]].append(e["t"])
    g1 = [.01517, .02022, .02527, .03037, .03547, .04057, .04567, .05077, .05587, .06092, .06597, .07102]
    g0 = [.01012, .02024, .03036, .04053, .04558, .05063, .05568, .06073, .06578]
    assert np.allclose(ends[1], g1, atol=1e-12, rtol=0) and np.allclose(ends[0], g0, atol=1e-12, rtol=0)
    assert int(st["placed_solo"][0, 0]) == 3 and int(st["placed_mixed"][0, 0]) == 1
    tpot = .005075 + (.05587 - .02024) / 6 + (.06578 - .03036) / 6 + (.07102 - .04053) / 6
    assert abs(st["sum_tpot"][0, 0] - tpot) < 1e-12
    # the decode buffer held d for 0.00004 s
    assert abs(st["area_Qd"][0, 0] - 0.00004) < 1e-12


@pytest.mark.parametrize("chunk,expected_iters", [(256, 3), (512, 2), (1024, 1), (100, 6)])
def test_chunked_prefill_takes_ceil_P_over_C_iterations(chunk, expected_iters):
    # Section 2.3: a prefill of P tokens advances C tokens per iteration
    inp = presets.single_class(N=1, B=2, C=chunk, P=600, D=1, M=1, inject=[(0.0, 0, 600, 1)])
    tr, st, _ = _trace(inp, 50)
    pf = [e for e in tr if e["type"] == "PREFILL_DONE"][0]
    iters_before = [e for e in tr if e["type"] == "ITER_END" and e["t"] <= pf["t"]]
    assert len(iters_before) == expected_iters
    full, last = divmod(600, chunk)
    t = (0.005 + 2e-5 * chunk) * full + ((0.005 + 2e-5 * last) if last else 0.0)
    assert abs(pf["t"] - t) < 1e-12
