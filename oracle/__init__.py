"""CPU oracle of the gate-and-route simulation.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs may import this
package.  It shares nothing with the CUDA library: its own C source, its own ctypes layouts.
"""
from .qsim_oracle import OracleSim, bin_lower_edge, build_oracle, hist_percentiles, lib, run_oracle  # noqa: F401
from .ctmc_oracle import CtmcOracle, build_ctmc_oracle, ctmc_revenue_rate, run_ctmc_oracle  # noqa: F401,E402
