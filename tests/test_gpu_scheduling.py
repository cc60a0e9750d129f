"""How the replications are laid over the device does not change any result: launches that run the horizon in chunks per
replication (one block per resident slot, units handed out through a counter) against plain launches of one block per
replication, and the one-thread-per-replication kernels at 4, 8 and 32 replications per warp.  Every integer statistic and
the per-GPU end state must be identical bit for bit (fp64 sums to 1e-9), also when the event budget stops replications in mid-chunk and when a
checkpoint taken after a chunked run is resumed by a new handle.  Parity of the plain launches with the CPU oracle is
covered by the other GPU tests; one case here is checked against the oracle directly."""
import contextlib
import os

import numpy as np
import pytest
import torch

from qsim_inputs import presets

from parity import assert_parity

pytestmark = pytest.mark.gpu


@contextlib.contextmanager
def env(**kv):
    keep = {k: os.environ.get(k) for k in kv}
    for k, v in kv.items():
        if v is None:
            os.environ.pop(k, None)
        else:
            os.environ[k] = str(v)
    try:
        yield
    finally:
        for k, v in keep.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


def run(inp, horizons, budget=None, states=3, **kv):
    from paper_2602_02987_b200 import QSim
    with env(**kv):
        sim = QSim(inp)
        if budget:
            sim.set_event_budget(budget)
        for h in horizons:
            sim.run(h)
        st = sim.stats()
        launches = sim.launch_count()
        state = [sim.server_state(r) for r in range(min(inp.R, states))]
        info = sim.layout_info()
        sim.close()
    return st, state, launches, info


def same(a, b, what):
    """Integer statistics and the end state bit for bit; fp64 sums within 1e-9 relative (a launch adds the sums of its
    finished requests to the totals when it ends, so chunks change the order of those additions)."""
    assert_parity(a[0], b[0], what=what)
    for x, y in zip(a[1], b[1]):
        for k in x:
            assert np.array_equal(x[k], y[k]), (what, "GPU state", k)


@pytest.mark.parametrize("make,horizon", [
    (lambda: presets.cfg4(N=16, R=40, horizon_iters=600), 600),
    (lambda: presets.cfg2(N=96, R=7, horizon_iters=400), 400),
    (lambda: presets.cfg3(N=96, R=5, block_len=1.0), 700),
    (lambda: presets.cfg1(R=6), 900),
])
def test_chunked_launches_equal_plain_launches(make, horizon):
    inp = make()
    plain = run(inp, [horizon], QSIM_FAMILY="warp", QSIM_CHUNKS=1)
    for K in (2, 5, 16):
        got = run(inp, [horizon], QSIM_FAMILY="warp", QSIM_CHUNKS=K)
        same(got, plain, f"{inp.name}: {K} chunks")
    # several calls, each in chunks
    got = run(inp, [horizon // 3, horizon - horizon // 3], QSIM_FAMILY="warp", QSIM_CHUNKS=3)
    same(got, plain, f"{inp.name}: two calls of 3 chunks")


def test_chunked_launches_with_several_warps_per_replication():
    inp = presets.cfg4(N=160, R=5, horizon_iters=300)
    plain = run(inp, [300], QSIM_FAMILY="warp", QSIM_WARPS=4, QSIM_CHUNKS=1)
    assert plain[3]["warps"] == 4
    got = run(inp, [300], QSIM_FAMILY="warp", QSIM_WARPS=4, QSIM_CHUNKS=4)
    same(got, plain, "4 warps per replication, 4 chunks")


def test_event_budget_stops_replications_in_mid_chunk():
    inp = presets.cfg4(N=16, R=24, horizon_iters=500)
    plain = run(inp, [500], QSIM_FAMILY="warp", QSIM_CHUNKS=1)
    got = run(inp, [500], budget=100, QSIM_FAMILY="warp", QSIM_CHUNKS=4)       # the budget counts look-ahead rounds
    same(got, plain, "4 chunks, 100 rounds per chunk and launch")
    assert got[2] >= plain[2] + 3         # the budget forced further launches


def test_more_replications_than_resident_blocks_are_chunked_by_default():
    """2000 small replications on a device that holds fewer blocks: the library chunks on its own."""
    from paper_2602_02987_b200 import QSim
    inp = presets.cfg4(N=16, R=2000, horizon_iters=200)
    plain = run(inp, [200], QSIM_FAMILY="warp", QSIM_CHUNKS=1)
    auto = run(inp, [200], QSIM_FAMILY="warp", QSIM_CHUNKS=None)
    same(auto, plain, "automatic chunks")
    # and three sampled replications against the oracle
    from oracle import OracleSim
    for r in (0, 777, 1999):
        o = OracleSim(inp.with_(R=1, rep_offset=inp.rep_offset + r))
        o.run(200)
        ref = o.stats()
        o.close()
        for k in ("arrivals", "admitted", "prefill_done", "done_mixed", "done_solo", "abandoned_p", "abandoned_d", "iters_mixed", "iters_solo"):
            assert np.array_equal(np.asarray(auto[0][k][r]), np.asarray(ref[k][0])), (r, k)


def test_checkpoint_after_chunked_run_resumes_in_chunks():
    from paper_2602_02987_b200 import QSim
    inp = presets.cfg4(N=16, R=12, horizon_iters=400)
    whole = run(inp, [400, 300], QSIM_FAMILY="warp", QSIM_CHUNKS=1)
    with env(QSIM_FAMILY="warp", QSIM_CHUNKS=5):
        a = QSim(inp)
        a.run(400)
        saved = a.checkpoint()
        a.close()
        b = QSim(inp, checkpoint=saved)
        b.run(300)
        st = b.stats()
        state = [b.server_state(r) for r in range(3)]
        b.close()
    same((st, state), whole, "resumed in chunks")


@pytest.mark.parametrize("make,horizon", [
    (lambda: presets.cfg4(N=24, R=41, horizon_iters=500), 500),
    (lambda: presets.cfg2(N=96, R=9, horizon_iters=300), 300),
])
def test_replications_per_warp_do_not_matter(make, horizon):
    inp = make()
    base = run(inp, [horizon], QSIM_FAMILY="lane", QSIM_LANE_LSH=5)
    assert base[3]["warps"] == 0
    for lsh in (2, 3, 4):
        got = run(inp, [horizon], QSIM_FAMILY="lane", QSIM_LANE_LSH=lsh)
        same(got, base, f"{inp.name}: {1 << lsh} replications per warp")


@pytest.mark.parametrize("seed", range(8))
def test_random_configurations_in_chunks_against_the_oracle(seed):
    """The seeded random configurations of the fuzz test, run as launches of 3 and of 7 chunks per replication."""
    from oracle import OracleSim
    from test_gpu_fuzz import random_case
    inp = random_case(40 + seed)
    H = int(np.random.default_rng(seed).choice([300, 1500, 4000]))
    o = OracleSim(inp)
    o.run(H)
    ref = o.stats()
    ostate = [o.server_state(r) for r in range(inp.R)]
    o.close()
    for K in (3, 7):
        got = run(inp, [H // 2, H - H // 2], states=inp.R, QSIM_FAMILY="warp", QSIM_CHUNKS=K)
        same(got, (ref, ostate), f"{inp.name}: N={inp.N} B={inp.B} I={inp.I} router={inp.router}, {K} chunks")
