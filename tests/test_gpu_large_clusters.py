"""Parity of the several-warps instances (clusters of 512 simulated GPUs and more) with the CPU oracle in steady state:
horizons well past one decode lifetime, so that batches are full, requests finish, wait and abandon under every warp
count, at the cluster sizes of the benchmark configurations."""
import os
import threading

import numpy as np
import pytest

from qsim_inputs import presets
from qsim_inputs.spec import PLACE_LEAST_LOADED, PLACE_RANDOM, ROUTER_SLI

from parity import assert_parity

pytestmark = pytest.mark.gpu


def gpu_stats(inp, horizon, chunks=None, warps=None):
    from paper_2602_02987_b200 import QSim
    keep = os.environ.get("QSIM_WARPS")
    if warps is not None:
        os.environ["QSIM_WARPS"] = str(warps)
    try:
        sim = QSim(inp)
        if warps is not None:
            assert sim.layout_info()["warps"] == warps
        for h in (chunks or [horizon]):
            sim.run(h)
        st = sim.stats()
        state = [sim.server_state(r) for r in range(inp.R)]
        sim.close()
    finally:
        if warps is not None:
            if keep is None:
                del os.environ["QSIM_WARPS"]
            else:
                os.environ["QSIM_WARPS"] = keep
    return st, state


def oracle_stats(inp, horizon):
    """One oracle handle per replication, on threads (the C code runs without the interpreter lock)."""
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
    return st, [out[r][1] for r in range(inp.R)]


def check(inp, horizon, **kw):
    ref, rstate = oracle_stats(inp, horizon)
    got, gstate = gpu_stats(inp, horizon, **kw)
    assert_parity(got, ref, what=f"{inp.name} N={inp.N} {kw}")
    for a, b in zip(gstate, rstate):
        for k in a:
            assert np.array_equal(a[k], b[k]), (inp.name, "GPU state", k)
    return ref


@pytest.mark.parametrize("N,H", [(1024, 700), (4096, 450)])
def test_cfg4_steady_state_at_benchmark_cluster_sizes(N, H):
    # occupancy gate, SLI-aware router, histograms; four (N = 1024) and sixteen (N = 4096) warps per replication in the warp family
    st = check(presets.cfg4(N=N, R=2), H, chunks=[H // 3, H - H // 3])
    done = st["done_mixed"] + st["done_solo"]
    assert done.sum() > 20 * N and st["abandoned_p"].sum() > 0
    assert st["hist_tpot"].sum() == done.sum()


def test_cfg3_full_cluster_all_blocks_with_role_changes():
    # priority gate, 24 blocks, per-block targets: M changes at more than two block ends
    inp = presets.cfg3(N=1024, R=2, block_len=0.5)
    assert int((np.diff(inp.M.astype(int)) != 0).sum()) >= 2
    st = check(inp, inp.meta["horizon_iters"])
    assert st["abandoned_p"].sum() > 0 and (st["done_mixed"] + st["done_solo"]).sum() > 20_000


def test_cfg2_full_cluster_with_abandonment():
    st = check(presets.cfg2(N=512, R=2), 700)
    assert st["abandoned_p"].sum() > 0


@pytest.mark.parametrize("N,H,placement", [(1100, 1000, PLACE_RANDOM), (2100, 600, PLACE_LEAST_LOADED), (2100, 300, PLACE_RANDOM)])
def test_decode_backlog_on_large_clusters(N, H, placement):
    # decode slots scarce: thousands of requests wait in the decode buffer and abandon it, every decode completion
    # frees a slot that the buffer's head takes (solo GPUs first), on both sides of the eight-warp threshold
    st = check(presets.crowded("decode", N=N, R=2, placement=placement), H)
    assert st["abandoned_d"].sum() > 1000 and st["Qd"].sum() > 1000
    assert st["placed_solo"].sum() > 0 and st["placed_mixed"].sum() > 0


def test_prefill_backlog_with_the_sli_router_on_a_large_cluster():
    inp = presets.crowded("prefill", N=1500, R=2, placement=PLACE_LEAST_LOADED, router=ROUTER_SLI)
    st = check(inp, 800)
    assert st["abandoned_p"].sum() > 1000


@pytest.mark.parametrize("warps", [2, 4, 8, 16])
def test_every_warp_count_gives_the_same_trajectory(warps):
    # the number of warps per replication is a launch parameter, not part of the method
    for inp, H in ((presets.cfg4(N=640, R=2), 400), (presets.crowded("decode", N=530, R=2), 500),
                   (presets.cfg3(N=512, R=1, block_len=0.25), None)):
        check(inp, H or inp.meta["horizon_iters"], warps=warps)


def test_one_warp_instances_agree_on_a_cluster_that_defaults_to_several_warps():
    inp = presets.cfg2(N=1024, R=2)
    check(inp, 200, warps=1)


def test_handles_of_different_sizes_share_kernels():
    """A large handle stays usable after smaller handles of the same kernel instance were created and a call of the
    static-memory entry point ran in between (the kernels' shared-memory limit is per kernel, not per handle)."""
    from paper_2602_02987_b200 import QSim, simulate_static
    big_inp = presets.cfg4(N=4096, R=1)
    big = QSim(big_inp)
    big.run(20)
    small = QSim(presets.cfg4(N=1024, R=1))
    small.run(20)
    simulate_static(presets.cfg0(R=2, horizon_iters=200), 200)
    big.run(20)                                   # must still launch with its 200 KB of shared memory
    got = big.stats()
    big.close(); small.close()
    ref, _ = oracle_stats(big_inp, 40)
    assert_parity(got, ref, what="large handle after smaller ones")
