"""ctypes front end of the C oracle of the exponential-service model (ctmc_oracle.c).  TEST INFRASTRUCTURE ONLY.

`run_ctmc_oracle(inputs, T_end)` returns a dict of numpy arrays keyed by the statistic names of
`qsim_inputs.spec` (CTMC_COUNTERS, CTMC_STATE, CTMC_AREAS, "events", "T_elapsed").
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, n) for n in ("ctmc_oracle.c", "qsim_oracle.c")]
_HDRS = [os.path.join(_HERE, n) for n in ("ctmc_oracle.h", "qsim_oracle.h")]
_LIB = os.path.join(_HERE, "libctmc_oracle.so")

_COUNTERS = ("arrivals", "admitted", "prefill_done", "placed_mixed", "placed_solo", "done_mixed", "done_solo",
             "abandoned_p", "abandoned_d", "overflow_d")
_STATE = ("Qp", "X", "Qd", "Ym", "Ys")
_AREAS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys")


class Config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("I", "N", "M", "B", "R", "qcap", "gate", "router")] + \
               [("seed", C.c_uint64), ("rep_offset", C.c_uint64)]


class Class(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("lam", "theta", "mu_p", "mu_m", "mu_s", "xstar", "n_xstar", "n_qpstar",
                                          "p_solo")] + [("prio_rank", C.c_uint32), ("pad", C.c_uint32)]


class RepStats(C.Structure):
    _fields_ = [("cnt", (C.c_uint64 * len(_COUNTERS)) * 8), ("state", (C.c_uint32 * 5) * 8), ("pad", C.c_uint32 * 8),
                ("area", (C.c_double * 5) * 8), ("events", C.c_uint64), ("T_elapsed", C.c_double)]


def build_ctmc_oracle(force: bool = False) -> str:
    stale = (not os.path.exists(_LIB)) or any(os.path.getmtime(p) > os.path.getmtime(_LIB) for p in _SRCS + _HDRS)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", _LIB] + _SRCS + ["-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build_ctmc_oracle())
        L.ctmc_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config), C.POINTER(Class)]
        L.ctmc_run_until.argtypes = [C.c_void_p, C.c_double, C.c_uint32, C.c_uint32]
        L.ctmc_stats.argtypes = [C.c_void_p, C.c_void_p]
        L.ctmc_destroy.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def marshal(inp):
    cfg = Config(I=inp.I, N=inp.N, M=inp.M, B=inp.B, R=inp.R, qcap=inp.qcap, gate=inp.gate, router=inp.router,
                 seed=inp.seed, rep_offset=inp.rep_offset)
    classes = (Class * inp.I)()
    for i in range(inp.I):
        classes[i] = Class(lam=float(inp.lam[i]), theta=float(inp.theta[i]), mu_p=float(inp.mu_p[i]),
                           mu_m=float(inp.mu_m[i]), mu_s=float(inp.mu_s[i]), xstar=float(inp.xstar[i]),
                           n_xstar=float(inp.n_xstar[i]), n_qpstar=float(inp.n_qpstar[i]), p_solo=float(inp.p_solo[i]),
                           prio_rank=int(inp.prio_rank[i]), pad=0)
    return cfg, classes


def unpack(per, R, I) -> dict:
    out = {}
    for k, n in enumerate(_COUNTERS):
        out[n] = np.array([[per[r].cnt[i][k] for i in range(I)] for r in range(R)], np.uint64)
    for k, n in enumerate(_STATE):
        out[n] = np.array([[per[r].state[i][k] for i in range(I)] for r in range(R)], np.uint32)
    for k, n in enumerate(_AREAS):
        out[n] = np.array([[per[r].area[i][k] for i in range(I)] for r in range(R)], np.float64)
    out["events"] = np.array([per[r].events for r in range(R)], np.uint64)
    out["T_elapsed"] = np.array([per[r].T_elapsed for r in range(R)], np.float64)
    return out


class CtmcOracle:
    def __init__(self, inp):
        self.inp = inp
        cfg, classes = marshal(inp)
        self.h = C.c_void_p()
        rc = lib().ctmc_create(C.byref(self.h), C.byref(cfg), classes)
        if rc != 0:
            raise RuntimeError(f"ctmc_create failed: {rc}")

    def run_until(self, T_end: float, rep_lo: int = 0, rep_hi: int | None = None) -> None:
        rc = lib().ctmc_run_until(self.h, float(T_end), rep_lo, self.inp.R if rep_hi is None else rep_hi)
        if rc != 0:
            raise RuntimeError(f"ctmc_run_until failed: {rc}")

    def stats(self) -> dict:
        per = (RepStats * self.inp.R)()
        if lib().ctmc_stats(self.h, per) != 0:
            raise RuntimeError("ctmc_stats failed")
        return unpack(per, self.inp.R, self.inp.I)

    def close(self) -> None:
        if self.h:
            lib().ctmc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def run_ctmc_oracle(inp, T_end: float, rep_lo: int = 0, rep_hi: int | None = None) -> dict:
    sim = CtmcOracle(inp)
    sim.run_until(T_end, rep_lo, rep_hi)
    st = sim.stats()
    sim.close()
    return st


def ctmc_revenue_rate(inp, st: dict, separate=None) -> np.ndarray:
    """Per-GPU revenue rate of every replication from the oracle's integer counters: bundled charging credits
    c_p P_i + c_d D_i at decode completion (Eq. (21)-(22)); separate charging credits c_p P_i at prefill
    completion and c_d D_i at decode completion (Eq. (23))."""
    sep = inp.meta.get("separate", False) if separate is None else separate
    done = (st["done_mixed"] + st["done_solo"]).astype(float)
    pf = st["prefill_done"].astype(float) if sep else done
    rev = (inp.prices[0] * inp.P * pf + inp.prices[1] * inp.D * done).sum(axis=1)
    return rev / (inp.N * st["T_elapsed"])
