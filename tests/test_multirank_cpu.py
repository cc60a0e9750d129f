"""World-size-2 check (gloo, CPU) of the multi-GPU layout: replications sharded by rank, statistics
gathered in replication order.  Each rank runs its shard with the CPU oracle standing in for its GPU."""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, R, horizon, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import run_oracle
    from paper_2602_02987_b200.sharding import combine_totals, gather_stats, shard, totals
    from qsim_inputs import presets
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    count, offset = shard(R, world, rank)
    inp = presets.cfg0(R=count, horizon_iters=horizon).with_(rep_offset=offset)
    local = run_oracle(inp, horizon)
    everything = gather_stats(local)
    # the benchmark's end-of-run exchange: each rank's own totals and its time
    mine = {"iters": int(local["iters_mixed"].sum() + local["iters_solo"].sum()), "events": int(local["events"].sum()),
            "T": float(local["T_elapsed"].sum())}
    combined = combine_totals(mine, 100.0 + rank)
    if rank == 0:
        np.savez(os.path.join(out_dir, "gathered.npz"), **everything)
        np.savez(os.path.join(out_dir, "totals.npz"), **totals(everything))
        np.savez(os.path.join(out_dir, "combined.npz"), **{k: np.array(v) for k, v in combined.items()})
    dist.barrier()
    dist.destroy_process_group()


def _ctmc_worker(rank, world, port, R, T_end, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import run_ctmc_oracle
    from paper_2602_02987_b200.sharding import gather_stats, shard
    from qsim_inputs import presets
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    count, offset = shard(R, world, rank)
    inp = presets.ctmc_instance(n=12, R=count, router=1).with_(rep_offset=offset)
    everything = gather_stats(run_ctmc_oracle(inp, T_end))
    if rank == 0:
        np.savez(os.path.join(out_dir, "ctmc.npz"), **everything)
    dist.barrier()
    dist.destroy_process_group()


def test_shard_covers_all_replications_once():
    from paper_2602_02987_b200.sharding import shard
    for R in (0, 1, 7, 8, 1024, 1000):
        for world in (1, 2, 3, 8):
            blocks = [shard(R, world, r) for r in range(world)]
            assert sum(c for c, _ in blocks) == R
            pos = 0
            for c, o in blocks:
                assert o == pos
                pos += c
            assert max(c for c, _ in blocks) - min(c for c, _ in blocks) <= 1
    with pytest.raises(ValueError):
        shard(4, 2, 2)


def test_two_ranks_reproduce_the_single_process_run(tmp_path):
    from oracle import run_oracle
    from paper_2602_02987_b200.sharding import totals
    from qsim_inputs import presets
    R, horizon, port = 7, 600, 29517
    mp.spawn(_worker, args=(2, port, R, horizon, str(tmp_path)), nprocs=2, join=True)
    got = dict(np.load(tmp_path / "gathered.npz"))
    tot = dict(np.load(tmp_path / "totals.npz"))
    want = run_oracle(presets.cfg0(R=R, horizon_iters=horizon), horizon)
    for k in want:
        assert np.array_equal(got[k], want[k]), k
    wt = totals(want)
    for k in wt:
        assert np.array_equal(tot[k], wt[k]), k
    # the benchmark's exchange of per-rank totals: integers exact, time = the slowest rank
    comb = dict(np.load(tmp_path / "combined.npz"))
    assert int(comb["iters"]) == int(want["iters_mixed"].sum() + want["iters_solo"].sum())
    assert int(comb["events"]) == int(want["events"].sum())
    assert abs(float(comb["T"]) - float(want["T_elapsed"].sum())) <= 1e-12 * float(comb["T"])
    assert float(comb["max_ms"]) == 101.0


def test_two_ranks_reproduce_the_exponential_service_run(tmp_path):
    from oracle import run_ctmc_oracle
    from qsim_inputs import presets
    R, T_end, port = 5, 40.0, 29531
    mp.spawn(_ctmc_worker, args=(2, port, R, T_end, str(tmp_path)), nprocs=2, join=True)
    got = dict(np.load(tmp_path / "ctmc.npz"))
    want = run_ctmc_oracle(presets.ctmc_instance(n=12, R=R, router=1), T_end)
    for k in want:
        assert np.array_equal(got[k], want[k]), k
