#!/usr/bin/env python
"""Benchmark: simulated GPU-server-iterations per second.

Default workload: cfg2, the largest configuration that is resident whole on one GPU (four lognormal classes at 1.05 of
the fluid capacity, N = 512 simulated GPUs, B = 256, R = 4096 replications per GPU).  One step = one pass of the whole
hot path (arrivals, next-event selection, iteration completion, accounting, decode routing, prefill gate, abandonment
clocks, iteration starts, statistics reduction) over one batch: all R replications advance by `--horizon` iterations of
horizon.  Steps continue the same simulation after a warm-up of at least 2000 iterations of horizon, so the timed steps
run in steady state.

    python bench.py --gpus N --steps K --warmup W          (N > 1: launched under torchrun, one rank per GPU)
    python bench.py --impl reference ...                   (the CPU oracle, timed on the host cores)
    python bench.py --workload cfg1 | cfg0 | cfg3 | cfg4 --cluster N | ctmc      (the other configurations)

Prints one JSON line.  `value` is timed with CUDA events around qsim_run with all state resident in HBM; `e2e` is the
same metric through qsim_simulate with host buffers (tables copied in, totals copied out, device memory allocated and
freed inside the timed region).
"""
from __future__ import annotations

import argparse
import hashlib
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
N_SM, SCHEDULERS = 148, 4  # issue peak of the GPU: SMs x schedulers x one warp instruction per cycle x SM clock
PREWARM = 2000             # iterations of horizon before the warm-up steps (steady state)

# workload -> (replications per GPU, iterations of horizon per step)
DEFAULTS = {"cfg2": (4096, 500), "cfg1": (1024, 100_000), "cfg0": (16, 10_000), "cfg3": (2048, 300), "cfg4": (8192, 300)}
CSRC = os.path.join(ROOT, "paper_2602_02987_b200", "csrc")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def kernel_source_id() -> str:
    """Fingerprint of the kernel sources: profile counters are only quoted for the sources they were taken with."""
    h = hashlib.sha256()
    for name in sorted(os.listdir(CSRC)):
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(name.encode()); h.update(f.read())
    return h.hexdigest()[:16]


def profile_counters(key: str):
    """Counters of an ncu capture kept beside its summary under profiles/ (per simulated server-iteration, or per jump):
    None when there is no capture for this workload or the kernels changed since it was taken."""
    path = os.path.join(ROOT, "profiles", "counters.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f).get(key)
    if not rec or rec.get("kernel_source_id") != kernel_source_id():
        return None
    return rec


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


def make_inputs(workload: str, reps: int, horizon: int, cluster: int):
    from qsim_inputs import presets
    kw = {"N": cluster} if cluster else {}
    if workload == "cfg1":
        return presets.cfg1(R=reps)
    if workload == "cfg0":
        return presets.cfg0(R=reps, horizon_iters=horizon)
    if workload == "cfg3":
        return presets.cfg3(R=reps, block_len=1.0, **kw)      # 24 blocks of 1 s instead of one hour each
    return getattr(presets, workload)(R=reps, horizon_iters=horizon, **kw)


def describe(workload: str, inp, reps: int, horizon: int) -> str:
    what = {"cfg0": "2 fixed-length classes, occupancy gate, solo-first router, bundled pricing",
            "cfg1": "2 lognormal classes, priority gate, solo-first router, separate pricing",
            "cfg2": "4 lognormal classes at 1.05 of the fluid capacity, occupancy gate, solo-first router, abandonment, bundled pricing",
            "cfg3": "4 lognormal classes, 24 blocks of 1 s (sinusoidal demand, per-block LP targets), priority gate, histograms",
            "cfg4": "cfg2 workload under constrained-LP targets, SLI-aware router, histograms"}[workload]
    return (f"{workload}: {what}; N={inp.N} GPUs, B={inp.B}, C={inp.C}, least-loaded placement, R={reps} replications per GPU, "
            f"{horizon} iterations of horizon per step")


def oracle_sample(workload: str, inp):
    """Bounded sample of the workload for the CPU oracle: about 10-20 s of work for the host cores (the oracle scans
    every GPU at every event).  Returns (replications, iterations of horizon each)."""
    cores = os.cpu_count() or 1
    h_s = 50_000 if workload == "cfg1" else max(100, int(1.0e6 / inp.N))
    return 2 * cores, h_s, cores


def oracle_throughput(inp, horizon_iters: int, n_reps: int, n_threads: int):
    """The CPU oracle as it stands, one replication per thread (the C code runs without the interpreter lock).  Handles
    are created before the clock starts; the clock covers the simulation only."""
    from oracle import OracleSim, build_oracle
    build_oracle()
    sims = [OracleSim(inp.with_(R=1, rep_offset=inp.rep_offset + r)) for r in range(n_reps)]
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
            sims[r].run(horizon_iters)

    t0 = time.perf_counter()
    threads = [threading.Thread(target=work) for _ in range(min(n_threads, n_reps))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    dt = time.perf_counter() - t0
    for r, sim in enumerate(sims):
        st = sim.stats()
        iters[r] = int(st["iters_mixed"].sum() + st["iters_solo"].sum())
        sim.close()
    return sum(iters) / dt, sum(iters), dt


def run_reference(args):
    """The reference arm: the oracle on the host cores, on the same bounded sample as the `cpu_baseline` leg."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = make_inputs(args.workload, 1, args.horizon, args.cluster)
    n_reps, h_s, cores = oracle_sample(args.workload, inp)
    vals, ms = [], []
    for s in range(args.warmup + args.steps):
        v, iters, dt = oracle_throughput(inp.with_(rep_offset=s * n_reps), h_s, n_reps, cores)
        if s >= args.warmup:
            vals.append(v); ms.append(dt * 1e3)
    value = sum(vals) / len(vals)
    sample = f"{n_reps} replications x {h_s} iterations of horizon of {args.workload} per step, one per thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sum(ms) / len(ms), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(args.workload, inp, args.reps, args.horizon), "sample": sample},
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
    from paper_2602_02987_b200.sharding import combine_totals, shard
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
    sampler = ClockSampler(local)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    if rank == 0:
        sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        T += dT; sim.run_until(T)
    b.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    tot = combine_totals({"jumps": int(sim.stats()["events"].sum()) - ev0, "launches": int(sim.launches - l0)}, a.elapsed_time(b))
    if rank == 0:
        t_ms, jumps = tot["max_ms"], tot["jumps"]
        rate = jumps / (t_ms * 1e-3)
        prof = profile_counters("qsim_ctmc_kernel")
        issue_peak = N_SM * SCHEDULERS * (clocks["sm_mhz"] or 1965.0) * 1e6
        inst = prof["warp_inst_per_unit"] * rate / world if prof else None
        out = {"metric": "simulated jumps of the exponential-service model/sec", "value": rate,
               "unit": "jumps/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
               "ms_per_step": t_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": "f64", "data": "synthetic", "gpu_launches": tot["launches"], "clocks": clocks,
               # no memory or tensor roofline applies: the records are read and written once per launch; the kernel is
               # bound by instruction issue of dependent chains, so the fraction is taken against the issue peak
               "roofline": {"bound": "alu", "achieved": inst, "peak": issue_peak, "unit": "warp-inst/s",
                            "frac": inst / issue_peak if inst else None,
                            "traffic": prof["dram_bytes_per_launch"] if (prof and count == 37888 and world == 1 and dT == prof.get("seconds_per_launch")) else None,
                            "counters": "profiles/counters.json" if prof else "no capture for the current kernel sources"},
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
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg1", "ctmc", "cfg0", "cfg3", "cfg4"],
                    help="cfg2 (default): the largest configuration resident whole on one GPU; cfg1 / cfg0 / cfg3 / cfg4: the "
                         "other configurations (--cluster gives the simulated GPUs of cfg2-4); ctmc: the exponential-service "
                         "model, reported in jumps/s")
    ap.add_argument("--horizon", type=int, default=0, help="iterations of horizon per step (0 = the workload's default)")
    ap.add_argument("--reps", type=int, default=0, help="replications per GPU (0 = the workload's default)")
    ap.add_argument("--cluster", type=int, default=0, help="simulated GPUs per replication for cfg2 / cfg3 / cfg4 (0 = the preset's)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ctmc-seconds", type=float, default=10.0, help="simulated seconds per step of the ctmc workload")
    args = ap.parse_args()
    if args.workload == "ctmc":
        if args.impl == "reference":
            raise SystemExit("the reference arm times the iteration-level workloads")
        run_ctmc(args)
        return
    d_reps, d_h = DEFAULTS[args.workload]
    args.reps = args.reps or d_reps
    args.horizon = args.horizon or d_h
    if args.impl == "reference":
        run_reference(args)
        return
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist
    from paper_2602_02987_b200 import QSim, simulate_host
    from paper_2602_02987_b200.sharding import combine_totals, shard

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
    count, offset = shard(args.reps * world, world, rank)
    inp = make_inputs(args.workload, count, args.horizon, args.cluster).with_(rep_offset=offset)
    sim = QSim(inp, device=f"cuda:{local}")
    info = sim.layout_info()
    family = "one thread per replication" if info["warps"] == 0 else f"{info['warps']} warp(s) per replication"
    if args.workload not in ("cfg1", "cfg3"):
        sim.run(PREWARM)          # steady state before the warm-up steps (cfg1's steps are 10^5 iterations each; cfg3 is one day)
    for _ in range(args.warmup):
        sim.run(args.horizon)
    sim.reset_stats()             # the statistics below cover the timed region only
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
    launches = sim.launch_count() - launches0
    it1, ev1, tot1 = sim.totals()                 # reduced on the device: a few KB come back
    bundled, separate = sim.revenue(tot1)
    I = inp.I
    mine = {"iters": it1, "events": ev1, "launches": launches,
            "jobs": sum(int(tot1.cls[i].done_mixed + tot1.cls[i].done_solo) for i in range(I)),
            "overflow": sum(int(tot1.cls[i].overflow + tot1.cls[i].overflow_d) for i in range(I)),
            "abandoned": sum(int(tot1.cls[i].abandoned_p + tot1.cls[i].abandoned_d) for i in range(I)),
            "revenue_x_T": (separate if inp.pricing == 1 else bundled) * float(tot1.T_elapsed), "T": float(tot1.T_elapsed)}
    tot = combine_totals(mine, sum(step_ms))
    total_ms = tot["max_ms"]
    iters, events, jobs, n_launch = tot["iters"], tot["events"], tot["jobs"], tot["launches"]
    value = iters / (total_ms * 1e-3)

    # end to end through the host-buffer entry point (fresh system each step, totals reduced on the device)
    e2e = None
    if not args.no_e2e:
        h2d = int((inp.lengths.nbytes if inp.lengths is not None else 0) + inp.rates.nbytes + 8 * 6 + 8 * 2 + inp.nblk * 456 + inp.I * 24 + 80)
        d2h = 2048 + 8
        simulate_host(inp.with_(R=8), 50, per_rep=False)   # warm the context and allocator paths
        barrier()
        e_t, e_iters = 0.0, 0
        for _ in range(args.steps):
            t0 = time.perf_counter()
            st = simulate_host(inp, args.horizon, per_rep=False)["_totals"]
            e_t += time.perf_counter() - t0
            e_iters += int(st["iters_mixed"].sum() + st["iters_solo"].sum())
        et = combine_totals({"iters": e_iters}, e_t * 1e3)
        e2e = {"value": et["iters"] / (et["max_ms"] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "note": "fresh system each step (transient from empty, no warm-up): allocation, table upload, set-up, run, totals"}

    if rank == 0:
        peak, peak_kind = measured_peaks()
        # algorithmic HBM bytes of one launch of the dominant kernel (the run kernel): what the method must move is the
        # request life cycle; the warp-per-replication kernels also stage their per-GPU state once per launch
        stage = 2.0 * inp.R * (info["header_bytes"] + info["image_bytes"])
        n_l = max(n_launch / world, 1.0)
        alg_bytes_per_launch = (JOB_BYTES * jobs / world + stage * args.steps) / n_l
        kernel_ms = total_ms / n_l
        achieved = alg_bytes_per_launch / (kernel_ms * 1e-3) / 1e9
        key = f"{args.workload}:{'lane' if info['warps'] == 0 else 'warp'}" + (f":N{inp.N}" if args.cluster else "")
        prof = profile_counters(key)
        issue_peak = N_SM * SCHEDULERS * (clocks["sm_mhz"] or 1965.0) * 1e6
        lp_value = float(inp.meta["lp_value"][0]) if inp.nblk == 1 else None
        rev = tot["revenue_x_T"] / tot["T"] if tot["T"] > 0 else None
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(args.workload, inp, args.reps, args.horizon), "kernels": family,
                       "l2": "state larger than L2 (workspace %.0f MB per GPU)" % (sim.workspace_bytes / 1e6),
                       "prewarm_iterations": PREWARM if args.workload not in ("cfg1", "cfg3") else 0,
                       "events_per_iteration": events / iters, "requests_per_iteration": jobs / iters,
                       "queue_overflow": tot["overflow"], "abandoned": tot["abandoned"],
                       "revenue_per_gpu": rev, "lp_value": lp_value,
                       "revenue_over_lp": (rev / lp_value) if (rev is not None and lp_value) else None},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": prof["dram_bytes_per_unit"] * iters / world / n_l if prof else None,
                         "traffic_source": (f"ncu capture scaled by iterations ({prof['capture']})" if prof else
                                            "no capture for this workload with the current kernel sources"),
                         "peak_kind": peak_kind, "bytes_per_iteration": JOB_BYTES * jobs / iters,
                         "note": "latency/issue-bound event chains; the HBM fraction is the contract figure",
                         "issue": ({"achieved": prof["warp_inst_per_unit"] * value / world, "peak": issue_peak, "unit": "warp-inst/s",
                                    "frac": prof["warp_inst_per_unit"] * value / world / issue_peak} if prof else None)},
            "clocks": clocks, "gpu_launches": int(n_launch), "wall_s": wall,
        }
        if e2e:
            out["e2e"] = e2e
        if not args.no_cpu_baseline and world == 1:
            n_reps, h_s, cores = oracle_sample(args.workload, inp)
            v, it_s, dt = oracle_throughput(inp, h_s, n_reps, cores)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": f"{n_reps} replications x {h_s} iterations of horizon of {args.workload}, one per thread, {dt:.1f} s"}
        print(json.dumps(out))
    sim.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
