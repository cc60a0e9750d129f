"""Injected arrivals, time-based runs and target updates on the CUDA path: hand-worked trajectories and the
online-replanning trace replay, against the oracle and against the hand-computed totals."""
import numpy as np
import pytest

from qsim_inputs import online, presets

from parity import assert_parity

pytestmark = pytest.mark.gpu


def _both(inp, iters):
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    g = QSim(inp); g.run(iters); gs = g.stats(); gstate = g.server_state(0); g.close()
    o = OracleSim(inp); o.run(iters); os_ = o.stats(); ostate = o.server_state(0); o.close()
    assert_parity(gs, os_, what=inp.name)
    for k in gstate:
        assert np.array_equal(gstate[k], ostate[k]), k
    return gs


def test_hand_trajectory_one_gpu():
    # tests/golden/hand_trace_1gpu.txt: ttft 0.02024 + 0.03958, tpot 0.01017 + 0.00505, 6 iterations, revenue 1032
    inp = presets.single_class(N=1, B=3, C=256, P=512, D=2, M=1, inject=[(0.0, 0, 512, 2), (0.001, 0, 512, 2)])
    st = _both(inp, 20)
    assert abs(st["sum_ttft"][0, 0] - 0.05982) < 1e-12 and abs(st["sum_tpot"][0, 0] - 0.01522) < 1e-12
    assert int(st["iters_mixed"][0]) == 4 and int(st["iters_solo"][0]) == 2
    assert 1.0 * st["tokens_in_completed"].sum() + 2.0 * st["tokens_out_completed"].sum() == 1032.0
    assert abs(st["busy_mixed"][0] - 0.04058) < 1e-12 and abs(st["busy_solo"][0] - 0.0101) < 1e-12


def test_hand_trajectory_two_gpus():
    # tests/golden/hand_trace_2gpu.txt: three requests decode on the solo GPU, one on the mixed GPU, 0.00004 s of buffer wait
    inj = [(0.0, 0, 256, 6), (0.001, 0, 256, 6), (0.002, 0, 256, 6), (0.003, 0, 256, 6)]
    inp = presets.single_class(N=2, B=2, C=256, P=256, D=6, M=1, inject=inj)
    st = _both(inp, 40)
    assert int(st["placed_solo"][0, 0]) == 3 and int(st["placed_mixed"][0, 0]) == 1
    tpot = .005075 + (.05587 - .02024) / 6 + (.06578 - .03036) / 6 + (.07102 - .04053) / 6
    assert abs(st["sum_tpot"][0, 0] - tpot) < 1e-12
    assert abs(st["area_Qd"][0, 0] - 0.00004) < 1e-12
    assert int(st["iters_mixed"][0] + st["iters_solo"][0]) == 21


@pytest.mark.parametrize("placement", [0, 1])
def test_trace_replay_with_online_replanning(placement):
    from oracle import OracleSim
    from paper_2602_02987_b200 import QSim
    inp, Pm, Dm = presets.trace_replay(R=3, T=60.0, placement=placement)
    g = QSim(inp)
    dg = online.run_online(g, inp, Pm, Dm, 60.0)
    gs = g.stats(); g.close()
    o = OracleSim(inp)
    do = online.run_online(o, inp, Pm, Dm, 60.0)
    os_ = o.stats(); o.close()
    assert dg == do and len(dg) == 5
    assert_parity(gs, os_, what=f"trace replay, placement {placement}")
    assert gs["arrivals"][0].sum() == inp.inject_t.shape[0]


def test_run_until_matches_iteration_horizon_on_the_gpu():
    from paper_2602_02987_b200 import QSim
    inp = presets.cfg0(R=4, horizon_iters=800)
    a = QSim(inp); a.run(800); sa = a.stats(); a.close()
    b = QSim(inp); b.run_until(float(sa["T_elapsed"][0]) * 0.4); b.run_until(float(sa["T_elapsed"][0])); sb = b.stats(); b.close()
    for k in sa:
        if sa[k].dtype.kind == "f":
            assert np.allclose(sa[k], sb[k], rtol=1e-12, atol=0), k
        else:
            assert np.array_equal(sa[k], sb[k]), k
