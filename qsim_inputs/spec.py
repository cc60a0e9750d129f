"""Plain-data description of one simulation instance.

This module holds no simulation arithmetic.  It only fixes the names, enums and
array shapes of the inputs that both the CPU oracle wrapper and the CUDA binding
marshal into their own C structures, and the names of the statistics they return.

Notation follows the paper: I classes, n = N GPUs, B decode cap per GPU, C prefill
chunk size, (P_i, D_i) prompt/output lengths, lambda_i per-GPU arrival rates,
theta_i patience rates, (c_p, c_d) token prices, x*_i / q*_p,i / y*_m,i / y*_s,i the
steady-state LP targets, M the number of mixed GPUs.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

MAXI = 8          # max number of classes
LMAX = 8192       # max token length; length tables hold LMAX-1 thresholds per (class, kind)
NBIN = 1024       # bins of the log-linear latency histograms (32 octaves x 32 sub-bins)

# prefill gate
GATE_OCCUPANCY = 0   # occupancy-deviation gate (Section 4.1, "Upstream (prefill) gate")
GATE_PRIORITY = 1    # largest D_i/P_i first (Section 5.1.1, Prioritize-and-Route)
GATE_FCFS = 2        # oldest waiting request first, no class rule (ablation FG-SP of the EC ablation study)
# decode router
ROUTER_SOLO_FIRST = 0      # single FCFS buffer, solo GPUs first (Section 4.1, "Downstream routing")
ROUTER_SLI = 1             # randomized split with p_s,i, two buffers (Section 5.2)
ROUTER_SLI_GENERAL = 2     # as ROUTER_SLI, plus class selection inside each pool by the weights varpi (EC, General SLI-aware Extension)
ROUTER_IMMEDIATE = 3       # no router: a request decodes on the GPU that prefilled it, in the slot it holds (ablations FI-WSP / GI-WSP of the EC ablation study)
# choice of GPU inside the eligible set
PLACE_RANDOM = 0           # uniformly at random (paper)
PLACE_LEAST_LOADED = 1     # fewest decodes, lowest index on ties
# revenue that is reported as "the" revenue (both are always computed)
PRICING_BUNDLED = 0        # Eq. (21)-(22)
PRICING_SEPARATE = 1       # Eq. (23)
# request lengths
LENGTH_FIXED = 0           # every class-i request has (P_i, D_i)
LENGTH_TABLE = 1           # integer lengths drawn through per-class threshold tables


@dataclass
class SimInputs:
    """Everything a simulator needs; arrays are C-contiguous numpy arrays."""
    name: str
    I: int
    N: int
    R: int
    B: int
    C: int
    nblk: int = 1
    gate: int = GATE_OCCUPANCY
    router: int = ROUTER_SOLO_FIRST
    placement: int = PLACE_RANDOM
    pricing: int = PRICING_BUNDLED
    length_mode: int = LENGTH_FIXED
    qcap: int = 4096            # capacity (entries) of each per-class prefill queue and of each decode buffer
    hist: int = 0               # 1: record TTFT / TPOT histograms
    seed: int = 0
    rep_offset: int = 0         # global index of replication 0 (sharding across handles / GPUs)
    block_len: float = 0.0      # seconds per block; ignored when nblk == 1
    # per class
    P: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint32))       # [I] fixed prompt length
    D: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint32))       # [I] fixed output length
    theta: np.ndarray = field(default_factory=lambda: np.zeros(0, np.float64))  # [I] patience rate (1/s)
    prio_rank: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint32))  # [I] 0 = served first
    rates: np.ndarray = field(default_factory=lambda: np.zeros((0, 0)))         # [nblk, I] per-GPU lambda_i
    lengths: Optional[np.ndarray] = None   # None or uint32 [I, 2, LMAX] thresholds (kind 0 = prompt, 1 = output)
    prices: np.ndarray = field(default_factory=lambda: np.zeros(2))             # (c_p, c_d)
    coeffs: np.ndarray = field(default_factory=lambda: np.zeros(6))             # alpha_m, beta, delta_m, alpha_s, delta_s, kappa
    # LP targets per block
    M: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint32))       # [nblk]
    xstar: np.ndarray = field(default_factory=lambda: np.zeros((0, 0)))         # [nblk, I]   x*_i
    n_xstar: np.ndarray = field(default_factory=lambda: np.zeros((0, 0)))       # [nblk, I]   n x*_i
    n_qpstar: np.ndarray = field(default_factory=lambda: np.zeros((0, 0)))      # [nblk, I]   n q*_p,i
    p_solo: np.ndarray = field(default_factory=lambda: np.zeros((0, 0)))        # [nblk, I]   p_s,i
    w_solo: Optional[np.ndarray] = None    # [nblk, I] varpi_s,i  (class-selection weights of the general SLI router)
    w_mix: Optional[np.ndarray] = None     # [nblk, I] varpi_m,i
    # optional injected arrivals replacing the Poisson source (same list for every replication):
    # times [K] ascending, and (class, P, D) [K, 3]
    inject_t: Optional[np.ndarray] = None
    inject_job: Optional[np.ndarray] = None
    # free-form notes from the recipe (LP optimum, fluid capacity, class means ...); never read by a simulator
    meta: dict = field(default_factory=dict)

    def with_(self, **kw) -> "SimInputs":
        return replace(self, **kw)

    def validate(self) -> None:
        I, nblk = self.I, self.nblk
        assert 1 <= I <= MAXI and self.N >= 1 and self.R >= 1 and self.B >= 1 and self.C >= 1 and nblk >= 1
        assert self.P.shape == (I,) and self.D.shape == (I,) and self.theta.shape == (I,)
        assert self.prio_rank.shape == (I,)
        assert self.rates.shape == (nblk, I)
        assert self.prices.shape == (2,) and self.coeffs.shape == (6,)
        assert self.M.shape == (nblk,)
        for a in (self.xstar, self.n_xstar, self.n_qpstar, self.p_solo):
            assert a.shape == (nblk, I)
        if self.w_solo is None:
            self.w_solo = np.zeros((nblk, I))
        if self.w_mix is None:
            self.w_mix = np.zeros((nblk, I))
        assert self.w_solo.shape == (nblk, I) and self.w_mix.shape == (nblk, I)
        if self.length_mode == LENGTH_TABLE:
            assert self.lengths is not None and self.lengths.shape == (I, 2, LMAX)
            assert self.lengths.dtype == np.uint32
        if self.inject_t is not None:
            K = self.inject_t.shape[0]
            assert self.inject_t.dtype == np.float64 and self.inject_job.shape == (K, 3)
            assert self.inject_job.dtype == np.uint32 and np.all(np.diff(self.inject_t) >= 0)


# Names of the per-class integer counters every simulator returns (uint64 [R, I]).
CLASS_COUNTERS = (
    "arrivals",              # A_i
    "admitted",              # U_p,i
    "prefill_done",          # S_p,i
    "placed_mixed",          # U_dm,i
    "placed_solo",           # U_ds,i
    "done_mixed",            # S_dm,i
    "done_solo",             # S_ds,i
    "abandoned_p",           # B_p,i
    "abandoned_d",           # B_d,i
    "overflow",              # arrivals dropped because the bounded prefill queue was full (0 in conforming runs)
    "overflow_d",            # finished prefills dropped because the bounded decode buffer was full (0 likewise)
    "tokens_in_prefilled",   # sum of P over completed prefills
    "tokens_in_completed",   # sum of P over completed requests
    "tokens_out_completed",  # sum of D over completed requests
)
# Per-class end-of-run state (uint32 [R, I]).
CLASS_STATE = ("Qp", "X", "Qd", "Ym", "Ys")
# Per-class fp64 accumulators (float64 [R, I]).
CLASS_SUMS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys", "sum_ttft", "sum_tpot")
# Per-replication scalars.
REP_COUNTERS = ("iters_mixed", "iters_solo", "events")      # uint64 [R]
REP_SUMS = ("busy_mixed", "busy_solo", "T_elapsed")          # float64 [R]


# ---------------------------------------------------------------------------------------------
# Exponential-service (Markov chain) model of Section 2.3: plain data, no arithmetic.
# ---------------------------------------------------------------------------------------------
CTMC_COUNTERS = ("arrivals", "admitted", "prefill_done", "placed_mixed", "placed_solo", "done_mixed", "done_solo",
                 "abandoned_p", "abandoned_d", "overflow_d")      # uint64 [R, I]
CTMC_STATE = ("Qp", "X", "Qd", "Ym", "Ys")                       # uint32 [R, I] at the end time
CTMC_AREAS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys")   # float64 [R, I] time integrals


@dataclass
class CtmcInputs:
    """One instance of the exponential-service model: classes are described by rates, not lengths."""
    name: str
    I: int
    N: int
    M: int                      # mixed GPUs of the static partition
    B: int
    R: int
    gate: int = GATE_OCCUPANCY  # GATE_OCCUPANCY or GATE_PRIORITY
    router: int = ROUTER_SOLO_FIRST   # ROUTER_SOLO_FIRST or ROUTER_SLI
    qcap: int = 4096            # capacity of each decode buffer (entries)
    seed: int = 0
    rep_offset: int = 0
    lam: np.ndarray = field(default_factory=lambda: np.zeros(0))     # [I] per-GPU arrival rates lambda_i
    theta: np.ndarray = field(default_factory=lambda: np.zeros(0))   # [I] patience rates
    mu_p: np.ndarray = field(default_factory=lambda: np.zeros(0))    # [I] Eq. (4)
    mu_m: np.ndarray = field(default_factory=lambda: np.zeros(0))
    mu_s: np.ndarray = field(default_factory=lambda: np.zeros(0))
    P: np.ndarray = field(default_factory=lambda: np.zeros(0))       # [I] token lengths, for revenue only
    D: np.ndarray = field(default_factory=lambda: np.zeros(0))
    prices: np.ndarray = field(default_factory=lambda: np.zeros(2))  # (c_p, c_d)
    prio_rank: np.ndarray = field(default_factory=lambda: np.zeros(0, np.uint32))
    xstar: np.ndarray = field(default_factory=lambda: np.zeros(0))   # [I] x*_i
    n_xstar: np.ndarray = field(default_factory=lambda: np.zeros(0))
    n_qpstar: np.ndarray = field(default_factory=lambda: np.zeros(0))
    p_solo: np.ndarray = field(default_factory=lambda: np.zeros(0))
    meta: dict = field(default_factory=dict)

    def with_(self, **kw) -> "CtmcInputs":
        return replace(self, **kw)

    def validate(self) -> None:
        I = self.I
        assert 1 <= I <= MAXI and self.N >= 1 and 0 <= self.M <= self.N and self.B >= 1 and self.R >= 1
        assert self.gate in (GATE_OCCUPANCY, GATE_PRIORITY) and self.router in (ROUTER_SOLO_FIRST, ROUTER_SLI)
        for a in (self.lam, self.theta, self.mu_p, self.mu_m, self.mu_s, self.P, self.D, self.xstar, self.n_xstar,
                  self.n_qpstar, self.p_solo, self.prio_rank):
            assert a.shape == (I,)
