"""ctypes front end of the C oracle (qsim_oracle.c).  TEST INFRASTRUCTURE ONLY.

`run_oracle(inputs, horizon_iters)` returns a dict of numpy arrays keyed by the statistic names
of `qsim_inputs.spec`; the CUDA binding returns the same keys so tests compare name by name.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qsim_oracle.c")
_HDR = os.path.join(_HERE, "qsim_oracle.h")
_LIB = os.path.join(_HERE, "libqsim_oracle.so")

MAXI, LMAX, NBIN = 8, 8192, 1024

_COUNTERS = ("arrivals", "admitted", "prefill_done", "placed_mixed", "placed_solo", "done_mixed", "done_solo",
             "abandoned_p", "abandoned_d", "overflow", "overflow_d", "tokens_in_prefilled",
             "tokens_in_completed", "tokens_out_completed")
_STATE = ("Qp", "X", "Qd", "Ym", "Ys")
_SUMS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys", "sum_ttft", "sum_tpot")

EV_NAMES = {1: "ARRIVAL", 2: "ADMIT", 3: "PREFILL_DONE", 4: "PLACE", 5: "DECODE_DONE", 6: "ABANDON_P",
            7: "ABANDON_D", 8: "ITER_END", 9: "BLOCK", 10: "OVERFLOW"}


class Config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("I", "N", "R", "B", "C", "nblk", "gate", "router", "placement",
                                           "pricing", "length_mode", "qcap", "hist", "n_inject")] + \
               [("seed", C.c_uint64), ("rep_offset", C.c_uint64), ("block_len", C.c_double)]


class Class(C.Structure):
    _fields_ = [("P", C.c_uint32), ("D", C.c_uint32), ("prio_rank", C.c_uint32), ("pad", C.c_uint32),
                ("theta", C.c_double)]


class Targets(C.Structure):
    _fields_ = [("M", C.c_uint32), ("pad", C.c_uint32), ("xstar", C.c_double * MAXI),
                ("n_xstar", C.c_double * MAXI), ("n_qpstar", C.c_double * MAXI), ("p_solo", C.c_double * MAXI),
                ("w_solo", C.c_double * MAXI), ("w_mix", C.c_double * MAXI)]


class ClassStats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in _COUNTERS] + [(n, C.c_uint32) for n in _STATE] + \
               [("pad", C.c_uint32)] + [(n, C.c_double) for n in _SUMS]


class RepStats(C.Structure):
    _fields_ = [("cls", ClassStats * MAXI), ("iters_mixed", C.c_uint64), ("iters_solo", C.c_uint64),
                ("events", C.c_uint64), ("busy_mixed", C.c_double), ("busy_solo", C.c_double),
                ("T_elapsed", C.c_double)]


class TraceRec(C.Structure):
    _fields_ = [("t", C.c_double), ("aux", C.c_double), ("job", C.c_uint64), ("type", C.c_int32),
                ("cls", C.c_int32), ("server", C.c_int32), ("rep", C.c_int32)]


def compile_oracle(src: str, out: str) -> str:
    """gcc command of the oracle: every fp operation stays a single rounded IEEE double operation."""
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-I", _HERE, "-o", out, src, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return out


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc when its source is newer than the library."""
    stale = (not os.path.exists(_LIB)) or any(os.path.getmtime(p) > os.path.getmtime(_LIB) for p in (_SRC, _HDR))
    if force or stale:
        compile_oracle(_SRC, _LIB)
    return _LIB


_lib = None


def load_oracle(path: str):
    """Load an oracle library and declare its entry points (tests load deliberately broken copies this way)."""
    if True:
        L = C.CDLL(path)
        L.orc_create.restype = C.c_int
        L.orc_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config), C.POINTER(Class), C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(Targets), C.c_void_p, C.c_void_p]
        L.orc_set_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.orc_trace_count.restype = C.c_uint64
        L.orc_trace_count.argtypes = [C.c_void_p]
        L.orc_run.restype = C.c_int
        L.orc_run.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32]
        L.orc_reset_stats.argtypes = [C.c_void_p]
        L.orc_run_until.restype = C.c_int
        L.orc_run_until.argtypes = [C.c_void_p, C.c_double, C.c_uint32, C.c_uint32]
        L.orc_set_targets.restype = C.c_int
        L.orc_set_targets.argtypes = [C.c_void_p, C.POINTER(Targets)]
        L.orc_stats.restype = C.c_int
        L.orc_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_server_state.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_philox4x32_10.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.orc_qlog.restype = C.c_double
        L.orc_qlog.argtypes = [C.c_double]
        L.orc_u53.restype = C.c_double
        L.orc_u53.argtypes = [C.c_uint32, C.c_uint32]
        L.orc_tau.restype = C.c_double
        L.orc_tau.argtypes = [C.POINTER(C.c_double), C.c_uint32, C.c_uint32, C.c_uint64]
        L.orc_table_length.restype = C.c_uint32
        L.orc_table_length.argtypes = [C.c_void_p, C.c_uint32]
        L.orc_hist_bin.restype = C.c_uint32
        L.orc_hist_bin.argtypes = [C.c_double]
    return L


def lib():
    global _lib
    if _lib is None:
        _lib = load_oracle(build_oracle())
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


class OracleSim:
    """One oracle handle for all R replications of a SimInputs."""

    def __init__(self, inp, trace_cap: int = 0):
        L = lib()
        self.inp = inp
        I, nblk = inp.I, inp.nblk
        n_inject = 0 if inp.inject_t is None else int(inp.inject_t.shape[0])
        cfg = Config(I=I, N=inp.N, R=inp.R, B=inp.B, C=inp.C, nblk=nblk, gate=inp.gate, router=inp.router,
                     placement=inp.placement, pricing=inp.pricing, length_mode=inp.length_mode, qcap=inp.qcap,
                     hist=inp.hist, n_inject=n_inject, seed=inp.seed, rep_offset=inp.rep_offset,
                     block_len=inp.block_len)
        classes = (Class * I)()
        for i in range(I):
            classes[i] = Class(P=int(inp.P[i]), D=int(inp.D[i]), prio_rank=int(inp.prio_rank[i]), pad=0,
                               theta=float(inp.theta[i]))
        tg = (Targets * nblk)()
        for b in range(nblk):
            tg[b].M = int(inp.M[b])
            for i in range(I):
                tg[b].xstar[i] = float(inp.xstar[b, i])
                tg[b].n_xstar[i] = float(inp.n_xstar[b, i])
                tg[b].n_qpstar[i] = float(inp.n_qpstar[b, i])
                tg[b].p_solo[i] = float(inp.p_solo[b, i])
                if inp.w_solo is not None:
                    tg[b].w_solo[i] = float(inp.w_solo[b, i])
                    tg[b].w_mix[i] = float(inp.w_mix[b, i])
        rates = np.ascontiguousarray(inp.rates, np.float64)
        lengths = None if inp.lengths is None else np.ascontiguousarray(inp.lengths, np.uint32)
        prices = np.ascontiguousarray(inp.prices, np.float64)
        coeffs = np.ascontiguousarray(inp.coeffs, np.float64)
        inj_t = None if n_inject == 0 else np.ascontiguousarray(inp.inject_t, np.float64)
        inj_job = None if n_inject == 0 else np.ascontiguousarray(inp.inject_job, np.uint32)
        h = C.c_void_p()
        rc = L.orc_create(C.byref(h), C.byref(cfg), classes, _ptr(rates), _ptr(lengths), _ptr(prices),
                          _ptr(coeffs), tg, _ptr(inj_t), _ptr(inj_job))
        if rc != 0:
            raise RuntimeError(f"orc_create failed: {rc}")
        self.h = h
        self._trace = None
        if trace_cap:
            self._trace = (TraceRec * trace_cap)()
            L.orc_set_trace(self.h, self._trace, trace_cap)

    def run(self, horizon_iters: int, rep_lo: int = 0, rep_hi: int | None = None) -> None:
        rc = lib().orc_run(self.h, int(horizon_iters), rep_lo, self.inp.R if rep_hi is None else rep_hi)
        if rc != 0:
            raise RuntimeError(f"orc_run failed: {rc}")

    def run_until(self, T: float) -> None:
        rc = lib().orc_run_until(self.h, float(T), 0, self.inp.R)
        if rc != 0:
            raise RuntimeError(f"orc_run_until failed: {rc}")

    def set_targets(self, M, xstar, n_xstar, n_qpstar, p_solo, w_solo=None, w_mix=None) -> None:
        tg = Targets()
        tg.M = int(M)
        for i in range(self.inp.I):
            tg.xstar[i] = float(xstar[i]); tg.n_xstar[i] = float(n_xstar[i])
            tg.n_qpstar[i] = float(n_qpstar[i]); tg.p_solo[i] = float(p_solo[i])
            if w_solo is not None:
                tg.w_solo[i] = float(w_solo[i]); tg.w_mix[i] = float(w_mix[i])
        if lib().orc_set_targets(self.h, C.byref(tg)) != 0:
            raise RuntimeError("orc_set_targets failed")

    def reset_stats(self) -> None:
        lib().orc_reset_stats(self.h)

    def stats(self) -> dict:
        inp = self.inp
        R, I = inp.R, inp.I
        per = (RepStats * R)()
        ht = hp = None
        if inp.hist:
            ht = np.zeros((R, I, NBIN), np.uint64)
            hp = np.zeros((R, I, NBIN), np.uint64)
        rc = lib().orc_stats(self.h, per, _ptr(ht), _ptr(hp))
        if rc != 0:
            raise RuntimeError(f"orc_stats failed: {rc}")
        out = {}
        for n in _COUNTERS:
            out[n] = np.array([[getattr(per[r].cls[i], n) for i in range(I)] for r in range(R)], np.uint64)
        for n in _STATE:
            out[n] = np.array([[getattr(per[r].cls[i], n) for i in range(I)] for r in range(R)], np.uint32)
        for n in _SUMS:
            out[n] = np.array([[getattr(per[r].cls[i], n) for i in range(I)] for r in range(R)], np.float64)
        for n in ("iters_mixed", "iters_solo", "events"):
            out[n] = np.array([getattr(per[r], n) for r in range(R)], np.uint64)
        for n in ("busy_mixed", "busy_solo", "T_elapsed"):
            out[n] = np.array([getattr(per[r], n) for r in range(R)], np.float64)
        if inp.hist:
            out["hist_ttft"] = ht
            out["hist_tpot"] = hp
        return out

    def server_state(self, r: int) -> dict:
        N = self.inp.N
        n_dec = np.zeros(N, np.uint32); it = np.zeros(N, np.uint32)
        t_next = np.zeros(N, np.float64); pf_rem = np.zeros(N, np.uint32)
        lib().orc_server_state(self.h, r, _ptr(n_dec), _ptr(it), _ptr(t_next), _ptr(pf_rem))
        return dict(n_dec=n_dec, it=it, t_next=t_next, pf_rem=pf_rem)

    def trace(self) -> list:
        n = int(lib().orc_trace_count(self.h))
        if self._trace is None:
            return []
        n = min(n, len(self._trace))
        return [dict(t=e.t, aux=e.aux, job=int(e.job), type=EV_NAMES[e.type], cls=e.cls, server=e.server, rep=e.rep)
                for e in self._trace[:n]]

    def trace_overflowed(self) -> bool:
        return self._trace is not None and int(lib().orc_trace_count(self.h)) > len(self._trace)

    def close(self) -> None:
        if self.h:
            lib().orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bin_lower_edge(b):
    """Smallest latency (seconds) that falls into histogram bin b: the double whose top 17 bits are b + ((1023-20) << 5)."""
    bits = (np.asarray(b, np.uint64) + np.uint64((1023 - 20) << 5)) << np.uint64(47)
    return bits.view(np.float64)


def hist_percentiles(hist, q) -> np.ndarray:
    """Percentiles of a latency histogram [R, I, NBIN] pooled over replications: for class i and quantile q the lower
    edge of the first bin whose cumulative count reaches ceil(q * total); NaN without samples.  Returns [I, len(q)]."""
    pooled = hist.sum(axis=0).astype(np.int64)               # [I, NBIN]
    out = np.full((pooled.shape[0], len(q)), np.nan)
    for i in range(pooled.shape[0]):
        total = int(pooled[i].sum())
        if total == 0:
            continue
        cum = np.cumsum(pooled[i])
        for k, qq in enumerate(q):
            need = min(max(int(np.ceil(qq * total)), 1), total)
            out[i, k] = bin_lower_edge(np.array([np.searchsorted(cum, need, side="left")]))[0]
    return out


def run_oracle(inp, horizon_iters: int, rep_lo: int = 0, rep_hi: int | None = None) -> dict:
    sim = OracleSim(inp)
    sim.run(horizon_iters, rep_lo, rep_hi)
    st = sim.stats()
    sim.close()
    return st


if __name__ == "__main__":
    build_oracle(force=True)
    print("built", _LIB, file=sys.stderr)
