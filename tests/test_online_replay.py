"""Trace replay with online replanning (Section 6.2): the host-side controller and the oracle's replay."""
import numpy as np

from oracle import OracleSim
from qsim_inputs import online, presets


def test_rate_estimate_eq45():
    # lambda_hat = max{rho N / (n W_bar), lambda_min}, W_bar = min{W, max{t, eps}}
    lam = online.estimate_rates([300, 0], [0, 0], n=10, t_k=10.0)
    assert np.allclose(lam, [3 * 300 / (10 * 10.0), 1e-6])
    lam = online.estimate_rates([900, 450], [300, 150], n=10, t_k=50.0)
    assert np.allclose(lam, [3 * 600 / (10 * 30.0), 3 * 300 / (10 * 30.0)])
    assert np.allclose(online.estimate_rates([5], [5], n=4, t_k=0.0), [1e-6])


def test_replay_feeds_every_arrival_once_and_replanning_moves_the_split():
    inp, Pm, Dm = presets.trace_replay(R=2, T=45.0)
    sim = OracleSim(inp)
    decisions = online.run_online(sim, inp, Pm, Dm, 45.0)
    st = sim.stats()
    sim.close()
    n_by_class = np.bincount(inp.inject_job[:, 0], minlength=2)
    assert np.array_equal(st["arrivals"][0], n_by_class) and np.array_equal(st["arrivals"][1], n_by_class)
    assert [t for t, _ in decisions] == [10.0, 20.0, 30.0, 40.0]
    # cold start plans for lambda_min (M = 1); the first estimate moves the split up (Eq. (46))
    assert inp.M[0] == 1 and decisions[0][1] > 1
    u = {k: v.astype(np.int64) for k, v in st.items() if v.dtype.kind in "ui"}
    assert np.array_equal(u["Qp"], u["arrivals"] - u["admitted"] - u["abandoned_p"] - u["overflow"])
    assert np.array_equal(u["Ym"] + u["Ys"], u["placed_mixed"] + u["placed_solo"] - u["done_mixed"] - u["done_solo"])
    # token counters follow the request-level lengths of the trace
    done = u["done_mixed"] + u["done_solo"]
    assert (u["tokens_out_completed"] > 0).all() and (done <= u["arrivals"]).all()


def test_run_until_and_iteration_horizon_agree_when_the_end_times_coincide():
    inp = presets.cfg0(R=2, horizon_iters=500)
    a = OracleSim(inp); a.run(500); sa = a.stats(); a.close()
    b = OracleSim(inp); b.run_until(float(sa["T_elapsed"][0])); sb = b.stats(); b.close()
    for k in sa:
        assert np.array_equal(sa[k], sb[k]), k
