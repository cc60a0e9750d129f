"""A small launch of the run kernel for profilers: a warm-up launch, then the launch to capture.

    python -m paper_2602_02987_b200.profile_case FAMILY PRESET R H N

FAMILY is `warp` or `lane` (the kernel family, see QSIM_FAMILY), PRESET a recipe of qsim_inputs.presets (cfg2, cfg4 ...),
R replications, H iterations of horizon in the captured launch, N simulated GPUs per replication.  Prints the iterations,
events and finished requests of the captured launch, which turn profiler counters into per-iteration figures.
"""
import os
import sys


def main(argv):
    fam, name, R, H, N = argv[0], argv[1], int(argv[2]), int(argv[3]), int(argv[4])
    os.environ["QSIM_FAMILY"] = fam
    from qsim_inputs import presets
    from . import QSim
    inp = getattr(presets, name)(R=R, horizon_iters=H, N=N)
    sim = QSim(inp, device="cuda:0")
    sim.run(600)
    sim.sync()
    it0, ev0, tot0 = sim.totals()
    sim.run(H)
    sim.sync()
    it1, ev1, tot1 = sim.totals()
    jobs = sum(int(tot1.cls[i].done_mixed + tot1.cls[i].done_solo) - int(tot0.cls[i].done_mixed + tot0.cls[i].done_solo)
               for i in range(inp.I))
    print("captured_launch iters", it1 - it0, "events", ev1 - ev0, "jobs", jobs, "workspace_GB", sim.workspace_bytes / 1e9,
          "info", sim.layout_info())
    sim.close()


if __name__ == "__main__":
    main(sys.argv[1:])
