#!/usr/bin/env python
"""Benchmark: simulated GPU-server-iterations per second on the two-class lognormal workload (cfg1).

One step = one pass of the whole hot path (arrivals, next-event selection, iteration completion,
accounting, decode routing, prefill gate, abandonment clocks, iteration starts, state staging) over one
batch: all R = 1024 replications of N = 64 simulated GPUs advance by 10^5 iterations of horizon.  Steps
continue the same simulation, so the timed steps run in steady state.

    python bench.py --gpus N --steps K --warmup W          (N > 1: launched under torchrun, one rank per GPU)
    python bench.py --impl reference ...                   (the CPU oracle, timed on the host cores)

Prints one JSON line.  `value` is timed with CUDA events around qsim_run with all state resident in HBM;
`e2e` is the same metric through qsim_simulate with host buffers (tables copied in, statistics copied out,
device memory allocated and freed inside the timed region).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "simulated GPU-server-iterations/sec"
UNIT = "server-iterations/s"
JOB_BYTES = 128            # algorithmic bytes per request life cycle: queue entry, prefill record, decode slot,
                           # decode-buffer pass, each written and read once at 32-byte sector granularity
# DRAM bytes per simulated server-iteration of qsim_run_kernel on cfg1, from an ncu capture of a 2000-iteration
# launch (dram__bytes_read.sum + dram__bytes_write.sum = 734.9 MB for 1.415e8 iterations); traffic grows with the
# iterations of a launch, so a full launch is that figure times its iterations
NCU_DRAM_BYTES_PER_ITER = 734.9e6 / 1.415e8
# warp instructions per simulated server-iteration of the same capture (smsp__inst_executed.sum = 3.224e10)
NCU_WARP_INST_PER_ITER = 3.224e10 / 1.415e8
# exponential-service kernel, capture of a 1-second launch at R = 37888: 4.238e9 warp instructions for 8.339e7 jumps and
# 160.5 MB + 191.4 MB of DRAM traffic (the replication records once, plus the counters and integrals that are added to in
# place; the latter grows with the simulated time, so a longer launch has no traffic figure)
NCU_CTMC_WARP_INST_PER_JUMP = 4.238e9 / 8.339e7
NCU_CTMC_DRAM_BYTES_PER_LAUNCH = 351.9e6
# issue peak of the GPU: 148 SMs x 4 schedulers x one warp instruction per cycle at the maximum SM clock
ISSUE_PEAK = 148 * 4 * 1.965e9
HORIZON = 100_000          # iterations of horizon per step (cfg1)
R_PER_GPU = 1024


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "200"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_throughput(inp, horizon_iters: int, n_reps: int, n_threads: int):
    """The CPU oracle as it stands, one replication per thread (the C code runs without the GIL)."""
    from oracle import OracleSim, build_oracle
    build_oracle()
    iters = [0] * n_reps
    nxt = [0]
    lock = threading.Lock()

    def work():
        while True:
            with lock:
                r = nxt[0]
                nxt[0] += 1
            if r >= n_reps:
                return
            sim = OracleSim(inp.with_(R=1, rep_offset=inp.rep_offset + r))
            sim.run(horizon_iters)
            st = sim.stats()
            iters[r] = int(st["iters_mixed"].sum() + st["iters_solo"].sum())
            sim.close()

    t0 = time.perf_counter()
    threads = [threading.Thread(target=work) for _ in range(min(n_threads, n_reps))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    dt = time.perf_counter() - t0
    return sum(iters) / dt, sum(iters), dt


def run_reference(args, workload):
    from qsim_inputs import presets
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    inp = presets.cfg1(R=R_PER_GPU)
    # bounded sample of the workload per step: one replication per core, 2000 iterations of horizon each
    h_sample, n_reps = 2000, cores
    vals, ms = [], []
    for s in range(args.warmup + args.steps):
        v, iters, dt = oracle_throughput(inp.with_(rep_offset=s * n_reps), h_sample, n_reps, cores)
        if s >= args.warmup:
            vals.append(v); ms.append(dt * 1e3)
    value = sum(vals) / len(vals)
    sample = f"{n_reps} replications x {h_sample} iterations of horizon of {workload} per step, one per thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sum(ms) / len(ms), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ctmc(args):
    """Second workload: the exponential-service model of Section 2.3 on the paper's two-class synthetic instance,
    n = 1000 GPUs, SLI-aware router, 37888 replications per GPU (one resident wave: 148 SMs x 8 blocks x 32 threads);
    one step advances every replication by 10 s."""
    import torch
    import torch.distributed as dist
    from paper_2602_02987_b200 import QSimCTMC
    from paper_2602_02987_b200.sharding import shard
    from qsim_inputs import presets
    from qsim_inputs.spec import ROUTER_SLI
    world = int(os.environ.get("WORLD_SIZE", "1")); rank = int(os.environ.get("RANK", "0")); local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the simulator has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    n, R, dT = 1000, 37888, args.ctmc_seconds
    count, offset = shard(R * world, world, rank)
    inp = presets.ctmc_instance(n=n, R=count, router=ROUTER_SLI).with_(rep_offset=offset)
    sim = QSimCTMC(inp, device=f"cuda:{local}")
    T = 0.0
    for _ in range(max(args.warmup, 3)):
        T += dT; sim.run_until(T)
    ev0 = int(sim.stats()["events"].sum()); l0 = sim.launches
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        T += dT; sim.run_until(T)
    b.record()
    torch.cuda.synchronize()
    my = torch.tensor([a.elapsed_time(b), float(int(sim.stats()["events"].sum()) - ev0), float(sim.launches - l0)], dtype=torch.float64, device="cuda")
    tmax = my[:1].clone()
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX); dist.all_reduce(my[1:], op=dist.ReduceOp.SUM)
    if rank == 0:
        out = {"metric": "simulated jumps of the exponential-service model/sec", "value": float(my[1]) / (float(tmax[0]) * 1e-3),
               "unit": "jumps/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
               "ms_per_step": float(tmax[0]) / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": "f64", "data": "synthetic", "gpu_launches": int(my[2]),
               # no memory or tensor roofline applies: the records are read and written once per launch; the kernel is
               # bound by instruction issue of dependent chains, so the fraction is taken against the issue peak
               "roofline": {"bound": "alu", "achieved": NCU_CTMC_WARP_INST_PER_JUMP * float(my[1]) / world / (float(tmax[0]) * 1e-3),
                            "peak": ISSUE_PEAK, "unit": "warp-inst/s",
                            "frac": NCU_CTMC_WARP_INST_PER_JUMP * float(my[1]) / world / (float(tmax[0]) * 1e-3) / ISSUE_PEAK,
                            "traffic": NCU_CTMC_DRAM_BYTES_PER_LAUNCH if (count == 37888 and world == 1 and dT == 1.0) else None},
               "config": {"workload": f"exponential-service model, paper synthetic instance, n={n}, SLI-aware router, "
                                      f"{R} replications per GPU, {dT} s of simulated time per step"}}
        if not args.no_cpu_baseline and world == 1:
            from oracle import run_ctmc_oracle
            cores = os.cpu_count() or 1
            done = [0] * cores
            T_cpu = 30_000.0      # about 10 s of work for the host cores

            def work(k):
                st = run_ctmc_oracle(inp.with_(R=1, rep_offset=k), T_cpu)
                done[k] = int(st["events"].sum())
            t0 = time.perf_counter()
            th = [threading.Thread(target=work, args=(k,)) for k in range(cores)]
            for t in th:
                t.start()
            for t in th:
                t.join()
            dt = time.perf_counter() - t0
            out["cpu_baseline"] = {"value": sum(done) / dt, "unit": "jumps/s", "cores": cores, "kind": "oracle",
                                   "sample": f"{cores} replications x {T_cpu:.0f} s of simulated time, one per thread, {dt:.1f} s"}
        print(json.dumps(out))
    sim.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="qsim", choices=["qsim", "reference"])
    ap.add_argument("--horizon", type=int, default=HORIZON, help="iterations of horizon per step")
    ap.add_argument("--reps", type=int, default=R_PER_GPU, help="replications per GPU")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="cfg1", choices=["cfg1", "ctmc", "cfg0", "cfg2", "cfg3", "cfg4"],
                    help="cfg1: the iteration-level benchmark (default); ctmc: the exponential-service model, reported in "
                         "jumps/s; cfg0 / cfg2 / cfg3 / cfg4: the other configurations (give --reps and --horizon, and "
                         "--cluster for the GPUs of cfg2-4), without the end-to-end leg")
    ap.add_argument("--cluster", type=int, default=0, help="simulated GPUs per replication for cfg2 / cfg3 / cfg4 (0 = the preset's)")
    ap.add_argument("--ctmc-seconds", type=float, default=10.0, help="simulated seconds per step of the ctmc workload")
    args = ap.parse_args()
    if args.workload == "ctmc":
        run_ctmc(args)
        return
    workload = (f"cfg1: 2 lognormal classes, N=64 GPUs, B=128, C=256, separate pricing, priority gate, solo-first "
                f"router, least-loaded placement, R={args.reps} replications per GPU, {args.horizon} iterations "
                f"of horizon per step")
    other = args.workload != "cfg1"
    if other:
        args.no_e2e = True
        workload = (f"{args.workload}" + (f" with N={args.cluster} GPUs" if args.cluster else "") +
                    f", R={args.reps} replications per GPU, {args.horizon} iterations of horizon per step")
    if args.impl == "reference":
        run_reference(args, workload)
        return
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist
    from paper_2602_02987_b200 import QSim, simulate_host
    from qsim_inputs import presets

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the simulator has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # replications are independent: rank k simulates global replications [k R, (k+1) R)  (weak scaling)
    from paper_2602_02987_b200.sharding import shard
    count, offset = shard(args.reps * world, world, rank)
    if args.workload == "cfg1":
        inp = presets.cfg1(R=count)
    elif args.workload == "cfg0":
        inp = presets.cfg0(R=count, horizon_iters=args.horizon)
    elif args.workload == "cfg3":
        inp = presets.cfg3(R=count, block_len=1.0, **({"N": args.cluster} if args.cluster else {}))
    else:
        inp = getattr(presets, args.workload)(R=count, horizon_iters=args.horizon, **({"N": args.cluster} if args.cluster else {}))
    inp = inp.with_(rep_offset=offset)
    sim = QSim(inp, device=f"cuda:{local}")
    info = sim.layout_info()
    for _ in range(args.warmup):
        sim.run(args.horizon)
    it0, ev0, tot0 = sim.totals()
    jobs0 = sum(int(tot0.cls[i].done_mixed + tot0.cls[i].done_solo) for i in range(inp.I))
    launches0 = sim.launch_count()
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    t_wall0 = time.perf_counter()
    for a, b in evs:
        a.record()
        sim.run(args.horizon)
        b.record()
    barrier()
    wall = time.perf_counter() - t_wall0
    clocks = sampler.stop() if rank == 0 else None
    step_ms = [a.elapsed_time(b) for a, b in evs]
    it1, ev1, tot1 = sim.totals()
    jobs1 = sum(int(tot1.cls[i].done_mixed + tot1.cls[i].done_solo) for i in range(inp.I))
    launches = sim.launch_count() - launches0
    overflow = sum(int(tot1.cls[i].overflow + tot1.cls[i].overflow_d) for i in range(inp.I))
    my = torch.tensor([sum(step_ms), float(it1 - it0), float(ev1 - ev0), float(jobs1 - jobs0), float(launches),
                       float(overflow)], dtype=torch.float64, device="cuda")
    tmax = my[:1].clone()
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        dist.all_reduce(my[1:], op=dist.ReduceOp.SUM)
    total_ms = float(tmax[0])
    iters, events, jobs, n_launch, ovf = (float(x) for x in my[1:])
    value = iters / (total_ms * 1e-3)

    # end to end through the host-buffer entry point (fresh system each step)
    e2e = None
    if not args.no_e2e:
        e_iters, e_t = 0.0, 0.0
        h2d = int(inp.lengths.nbytes + inp.rates.nbytes + 8 * 6 + 8 * 2 + inp.nblk * 264 + inp.I * 24 + 80)
        d2h = 0
        simulate_host(inp.with_(R=8), 200)   # warm the context and allocator paths
        barrier()
        for _ in range(args.steps):
            t0 = time.perf_counter()
            st = simulate_host(inp, args.horizon)
            e_t += time.perf_counter() - t0
            e_iters += float(st["iters_mixed"].sum() + st["iters_solo"].sum())
            d2h = inp.R * info["header_bytes"]
        ev = torch.tensor([e_t, e_iters], dtype=torch.float64, device="cuda")
        tm = ev[:1].clone()
        if world > 1:
            dist.all_reduce(tm, op=dist.ReduceOp.MAX)
            dist.all_reduce(ev[1:], op=dist.ReduceOp.SUM)
        e2e = {"value": float(ev[1]) / float(tm[0]), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h}

    if rank == 0:
        peak, peak_kind = measured_peaks()
        # algorithmic HBM bytes of one launch of the dominant kernel (qsim_run_kernel): the server state is
        # resident in shared memory, so what must move is the request life cycle plus the state staging
        stage = 2.0 * inp.R * (info["header_bytes"] + info["image_bytes"])
        alg_bytes_per_launch = (JOB_BYTES * jobs / world + stage * args.steps) / max(n_launch / world, 1.0)
        kernel_ms = total_ms / max(n_launch / world, 1.0)
        achieved = alg_bytes_per_launch / (kernel_ms * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload, "l2": "state larger than L2 (workspace %.0f MB per GPU)" % (sim.workspace_bytes / 1e6),
                       "events_per_iteration": events / iters, "requests_per_iteration": jobs / iters,
                       "queue_overflow": ovf},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None if other else NCU_DRAM_BYTES_PER_ITER * iters / world / max(n_launch / world, 1.0),
                         "traffic_source": "no capture for this workload" if other else "ncu capture of a 2000-iteration launch, scaled by iterations",
                         "peak_kind": peak_kind,
                         "bytes_per_iteration": JOB_BYTES * jobs / iters,
                         "note": "latency/issue-bound event chain; HBM fraction is the contract figure",
                         "issue": None if other else {"achieved": NCU_WARP_INST_PER_ITER * value / world, "peak": ISSUE_PEAK,
                                                      "unit": "warp-inst/s", "frac": NCU_WARP_INST_PER_ITER * value / world / ISSUE_PEAK}},
            "clocks": clocks, "gpu_launches": int(n_launch), "wall_s": wall,
        }
        if e2e:
            out["e2e"] = e2e
        if not args.no_cpu_baseline and world == 1:
            cores = os.cpu_count() or 1
            # about 10 s of work for the host cores: the oracle scans every GPU at every event
            h_s = 50_000 if not other else max(100, int(1.0e6 / inp.N))
            v, it_s, dt = oracle_throughput(inp, h_s, 2 * cores, cores)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": f"{2 * cores} replications x {h_s} iterations of horizon of {args.workload}, one per thread, {dt:.1f} s"}
        print(json.dumps(out))
    sim.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
