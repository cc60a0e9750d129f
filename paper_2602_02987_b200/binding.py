"""ctypes binding of libqsim.so with the same names as include/qsim.h (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from .build import LIB

MAXI, LMAX, NBIN = 8, 8192, 1024

_COUNTERS = ("arrivals", "admitted", "prefill_done", "placed_mixed", "placed_solo", "done_mixed", "done_solo",
             "abandoned_p", "abandoned_d", "overflow", "overflow_d", "tokens_in_prefilled",
             "tokens_in_completed", "tokens_out_completed")
_STATE = ("Qp", "X", "Qd", "Ym", "Ys")
_SUMS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys", "sum_ttft", "sum_tpot")

EXPORTS = ("qsim_create", "qsim_workspace_bytes", "qsim_bind", "qsim_run", "qsim_run_until", "qsim_set_injected",
           "qsim_set_targets", "qsim_set_event_budget", "qsim_sync",
           "qsim_stats", "qsim_reset_stats", "qsim_revenue", "qsim_server_state", "qsim_simulate", "qsim_simulate_waves",
           "qsim_simulate_static", "qsim_launch_count", "qsim_round_count", "qsim_layout_info", "qsim_destroy", "qsim_last_error",
           "qsim_ctmc_workspace_bytes", "qsim_ctmc_init", "qsim_ctmc_run_until", "qsim_ctmc_stats", "qsim_ctmc_revenue", "qsim_bind_restore", "qsim_latency_percentiles")


class QSimError(RuntimeError):
    pass


class qsim_config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("size", "I", "N", "R", "B", "C", "nblk", "gate", "router", "placement",
                                           "pricing", "length_mode", "qcap", "hist")] + \
               [("seed", C.c_uint64), ("rep_offset", C.c_uint64), ("block_len", C.c_double)]


class qsim_class(C.Structure):
    _fields_ = [("P", C.c_uint32), ("D", C.c_uint32), ("prio_rank", C.c_uint32), ("reserved", C.c_uint32),
                ("theta", C.c_double)]


class qsim_targets(C.Structure):
    _fields_ = [("M", C.c_uint32), ("reserved", C.c_uint32), ("xstar", C.c_double * MAXI),
                ("n_xstar", C.c_double * MAXI), ("n_qpstar", C.c_double * MAXI), ("p_solo", C.c_double * MAXI),
                ("w_solo", C.c_double * MAXI), ("w_mix", C.c_double * MAXI)]


class qsim_class_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in _COUNTERS] + [(n, C.c_uint32) for n in _STATE] + \
               [("reserved", C.c_uint32)] + [(n, C.c_double) for n in _SUMS]


class qsim_rep_stats(C.Structure):
    _fields_ = [("cls", qsim_class_stats * MAXI), ("iters_mixed", C.c_uint64), ("iters_solo", C.c_uint64),
                ("events", C.c_uint64), ("busy_mixed", C.c_double), ("busy_solo", C.c_double),
                ("T_elapsed", C.c_double)]


class qsim_ctmc_config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("size", "I", "N", "M", "B", "R", "qcap", "gate", "router", "reserved")] + \
               [("seed", C.c_uint64), ("rep_offset", C.c_uint64)]


class qsim_ctmc_class(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("lam", "theta", "mu_p", "mu_m", "mu_s", "xstar", "n_xstar", "n_qpstar",
                                          "p_solo")] + [("prio_rank", C.c_uint32), ("reserved", C.c_uint32)]


_CTMC_COUNTERS = ("arrivals", "admitted", "prefill_done", "placed_mixed", "placed_solo", "done_mixed", "done_solo",
                  "abandoned_p", "abandoned_d", "overflow_d")
_CTMC_AREAS = ("area_Qp", "area_X", "area_Qd", "area_Ym", "area_Ys")


class qsim_ctmc_rep_stats(C.Structure):
    _fields_ = [("cnt", (C.c_uint64 * 10) * MAXI), ("state", (C.c_uint32 * 5) * MAXI), ("reserved", C.c_uint32 * MAXI),
                ("area", (C.c_double * 5) * MAXI), ("events", C.c_uint64), ("T_elapsed", C.c_double)]


_lib = None


def load_library():
    """Load the in-tree libqsim.so; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise QSimError(f"{LIB} is missing: build it with `python -m paper_2602_02987_b200.build` "
                            "(there is no CPU fallback)")
        L = C.CDLL(LIB)
        vp = C.c_void_p
        L.qsim_create.argtypes = [C.POINTER(vp), C.POINTER(qsim_config), C.POINTER(qsim_class), vp, vp, vp, vp,
                                  C.POINTER(qsim_targets)]
        L.qsim_workspace_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
        L.qsim_bind.argtypes = [vp, vp, C.c_size_t, vp]
        L.qsim_bind_restore.argtypes = [vp, vp, C.c_size_t, vp]
        L.qsim_latency_percentiles.argtypes = [vp, vp, C.c_uint32, vp, vp]
        L.qsim_run.argtypes = [vp, C.c_uint64]
        L.qsim_run_until.argtypes = [vp, C.c_double]
        L.qsim_set_injected.argtypes = [vp, vp, vp, C.c_uint64]
        L.qsim_set_targets.argtypes = [vp, C.POINTER(qsim_targets)]
        L.qsim_set_event_budget.argtypes = [vp, C.c_uint64]
        L.qsim_sync.argtypes = [vp]
        L.qsim_stats.argtypes = [vp, vp, vp, vp, vp]
        L.qsim_reset_stats.argtypes = [vp]
        L.qsim_ctmc_workspace_bytes.argtypes = [C.POINTER(qsim_ctmc_config), C.POINTER(C.c_size_t)]
        L.qsim_ctmc_init.argtypes = [C.POINTER(qsim_ctmc_config), C.POINTER(qsim_ctmc_class), vp, C.c_size_t, vp]
        L.qsim_ctmc_run_until.argtypes = [C.POINTER(qsim_ctmc_config), C.POINTER(qsim_ctmc_class), vp, C.c_size_t, vp,
                                          C.c_double, C.POINTER(C.c_uint64)]
        L.qsim_ctmc_stats.argtypes = [C.POINTER(qsim_ctmc_config), vp, C.c_size_t, vp, vp]
        L.qsim_ctmc_revenue.argtypes = [C.POINTER(qsim_ctmc_config), vp, vp, vp, vp, C.c_int, vp]
        L.qsim_revenue.argtypes = [vp, vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.qsim_server_state.argtypes = [vp, C.c_uint32, vp, vp, vp, vp]
        L.qsim_simulate.argtypes = [C.POINTER(qsim_config), C.POINTER(qsim_class), vp, vp, vp, vp,
                                    C.POINTER(qsim_targets), C.c_uint64, vp, vp]
        L.qsim_simulate_waves.argtypes = [C.POINTER(qsim_config), C.POINTER(qsim_class), vp, vp, vp, vp,
                                          C.POINTER(qsim_targets), C.c_uint64, C.c_uint32, vp, vp, C.POINTER(C.c_uint32)]
        L.qsim_simulate_static.argtypes = [C.POINTER(qsim_config), C.POINTER(qsim_class), vp, vp, vp, vp,
                                           C.POINTER(qsim_targets), C.c_uint64, vp, vp, vp]
        L.qsim_launch_count.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.qsim_round_count.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.qsim_layout_info.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.qsim_destroy.argtypes = [vp]
        L.qsim_last_error.restype = C.c_char_p
        for n in EXPORTS:
            if n != "qsim_last_error":
                getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        raise QSimError(f"qsim error {rc}: {load_library().qsim_last_error().decode()}")


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def marshal(inp):
    """SimInputs -> the C structs and arrays of qsim_create (kept alive by the returned tuple)."""
    I, nblk = inp.I, inp.nblk
    cfg = qsim_config(size=C.sizeof(qsim_config), I=I, N=inp.N, R=inp.R, B=inp.B, C=inp.C, nblk=nblk,
                      gate=inp.gate, router=inp.router, placement=inp.placement, pricing=inp.pricing,
                      length_mode=inp.length_mode, qcap=inp.qcap, hist=inp.hist, seed=inp.seed,
                      rep_offset=inp.rep_offset, block_len=inp.block_len)
    classes = (qsim_class * I)()
    for i in range(I):
        classes[i] = qsim_class(P=int(inp.P[i]), D=int(inp.D[i]), prio_rank=int(inp.prio_rank[i]), reserved=0,
                                theta=float(inp.theta[i]))
    tg = (qsim_targets * nblk)()
    for b in range(nblk):
        tg[b].M = int(inp.M[b])
        for i in range(I):
            tg[b].xstar[i] = float(inp.xstar[b, i])
            tg[b].n_xstar[i] = float(inp.n_xstar[b, i])
            tg[b].n_qpstar[i] = float(inp.n_qpstar[b, i])
            tg[b].p_solo[i] = float(inp.p_solo[b, i])
            tg[b].w_solo[i] = float(inp.w_solo[b, i])
            tg[b].w_mix[i] = float(inp.w_mix[b, i])
    rates = np.ascontiguousarray(inp.rates, np.float64)
    lengths = None if inp.lengths is None else np.ascontiguousarray(inp.lengths, np.uint32)
    prices = np.ascontiguousarray(inp.prices, np.float64)
    coeffs = np.ascontiguousarray(inp.coeffs, np.float64)
    return cfg, classes, rates, lengths, prices, coeffs, tg


def _unpack(per, R, I, T_hist=None):
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
    return out


class QSim:
    """One handle of the CUDA library; the workspace is a torch tensor on the chosen device."""

    def __init__(self, inp, device="cuda:0", stream=None, checkpoint=None):
        """checkpoint: bytes of a workspace saved by `checkpoint()` of a handle with the same inputs; the run resumes there."""
        import torch
        if not torch.cuda.is_available():
            raise QSimError("no CUDA device: the simulator has no CPU path")
        self.L = load_library()
        self.inp = inp
        self.device = torch.device(device)
        self._keep = marshal(inp)
        cfg, classes, rates, lengths, prices, coeffs, tg = self._keep
        self.h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.L.qsim_create(C.byref(self.h), C.byref(cfg), classes, _ptr(rates), _ptr(lengths),
                                      _ptr(prices), _ptr(coeffs), tg))
            if getattr(inp, "inject_t", None) is not None:
                it = np.ascontiguousarray(inp.inject_t, np.float64)
                ij = np.ascontiguousarray(inp.inject_job, np.uint32)
                _check(self.L.qsim_set_injected(self.h, _ptr(it), _ptr(ij), it.shape[0]))
            nbytes = C.c_size_t()
            _check(self.L.qsim_workspace_bytes(self.h, C.byref(nbytes)))
            self.workspace_bytes = int(nbytes.value)
            self.ws = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.ws.data_ptr() + 255) & ~255
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self._base = base
            if checkpoint is None:
                _check(self.L.qsim_bind(self.h, C.c_void_p(base), self.workspace_bytes, C.c_void_p(self.stream.cuda_stream)))
            else:
                off = base - self.ws.data_ptr()
                if checkpoint.numel() != self.workspace_bytes:
                    raise QSimError("checkpoint size does not match this configuration")
                self.ws[off:off + self.workspace_bytes].copy_(checkpoint)
                _check(self.L.qsim_bind_restore(self.h, C.c_void_p(base), self.workspace_bytes,
                                                C.c_void_p(self.stream.cuda_stream)))

    def checkpoint(self):
        """The workspace bytes (a CPU uint8 tensor) after the work queued so far: pass them to QSim(..., checkpoint=)."""
        self.sync()
        off = self._base - self.ws.data_ptr()
        return self.ws[off:off + self.workspace_bytes].cpu()

    def latency_percentiles(self, q):
        """(ttft, tpot), each [I, len(q)] seconds: lower edge of the histogram bin where the cumulative count reaches q."""
        q = np.ascontiguousarray(q, np.float64)
        ttft = np.zeros((self.inp.I, q.shape[0])); tpot = np.zeros((self.inp.I, q.shape[0]))
        _check(self.L.qsim_latency_percentiles(self.h, _ptr(q), q.shape[0], _ptr(ttft), _ptr(tpot)))
        return ttft, tpot

    def set_event_budget(self, n: int) -> None:
        _check(self.L.qsim_set_event_budget(self.h, int(n)))

    def run(self, horizon_iters: int) -> None:
        _check(self.L.qsim_run(self.h, int(horizon_iters)))

    def run_until(self, T: float) -> None:
        _check(self.L.qsim_run_until(self.h, float(T)))

    def set_targets(self, M, xstar, n_xstar, n_qpstar, p_solo, w_solo=None, w_mix=None) -> None:
        tg = qsim_targets()
        tg.M = int(M)
        for i in range(self.inp.I):
            tg.xstar[i] = float(xstar[i]); tg.n_xstar[i] = float(n_xstar[i])
            tg.n_qpstar[i] = float(n_qpstar[i]); tg.p_solo[i] = float(p_solo[i])
            if w_solo is not None:
                tg.w_solo[i] = float(w_solo[i]); tg.w_mix[i] = float(w_mix[i])
        _check(self.L.qsim_set_targets(self.h, C.byref(tg)))

    def sync(self) -> None:
        _check(self.L.qsim_sync(self.h))

    def reset_stats(self) -> None:
        _check(self.L.qsim_reset_stats(self.h))

    def launch_count(self) -> int:
        n = C.c_uint64()
        _check(self.L.qsim_launch_count(self.h, C.byref(n)))
        return int(n.value)

    def layout_info(self) -> dict:
        out = (C.c_uint64 * 4)()
        _check(self.L.qsim_layout_info(self.h, out))
        return dict(header_bytes=int(out[0]), image_bytes=int(out[1]), smem_bytes=int(out[2]), warps=int(out[3]))

    def round_count(self) -> int:
        n = C.c_uint64()
        _check(self.L.qsim_round_count(self.h, C.byref(n)))
        return int(n.value)

    def stats(self, with_totals=False) -> dict:
        R, I = self.inp.R, self.inp.I
        per = (qsim_rep_stats * R)()
        tot = qsim_rep_stats()
        ht = hp = None
        if self.inp.hist:
            ht = np.zeros((R, I, NBIN), np.uint64)
            hp = np.zeros((R, I, NBIN), np.uint64)
        _check(self.L.qsim_stats(self.h, C.byref(tot), per, _ptr(ht), _ptr(hp)))
        out = _unpack(per, R, I)
        if self.inp.hist:
            out["hist_ttft"] = ht
            out["hist_tpot"] = hp
        if with_totals:
            b, s = C.c_double(), C.c_double()
            _check(self.L.qsim_revenue(self.h, C.byref(tot), C.byref(b), C.byref(s)))
            out["_totals"] = _unpack((tot,), 1, I)
            out["_revenue_bundled"] = b.value
            out["_revenue_separate"] = s.value
        return out

    def totals(self):
        """(server iterations, events) summed over replications, cheaply."""
        tot = qsim_rep_stats()
        _check(self.L.qsim_stats(self.h, C.byref(tot), None, None, None))
        return int(tot.iters_mixed + tot.iters_solo), int(tot.events), tot

    def revenue(self, tot):
        """(bundled, separate) revenue per GPU per second of a totals record, Eq. (22)-(23)."""
        b, s = C.c_double(), C.c_double()
        _check(self.L.qsim_revenue(self.h, C.byref(tot), C.byref(b), C.byref(s)))
        return b.value, s.value

    def server_state(self, r: int) -> dict:
        N = self.inp.N
        n_dec = np.zeros(N, np.uint32); it = np.zeros(N, np.uint32)
        t_next = np.zeros(N, np.float64); pf_rem = np.zeros(N, np.uint32)
        _check(self.L.qsim_server_state(self.h, r, _ptr(n_dec), _ptr(it), _ptr(t_next), _ptr(pf_rem)))
        return dict(n_dec=n_dec, it=it, t_next=t_next, pf_rem=pf_rem)

    def close(self) -> None:
        if getattr(self, "h", None):
            self.L.qsim_destroy(self.h)
            self.h = None
            self.ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def simulate_host(inp, horizon_iters: int, per_rep: bool = True) -> dict:
    """qsim_simulate: host buffers in, host statistics out (allocates and frees its own device memory).
    per_rep=False asks for the totals only: they are reduced on the device and a few KB come back."""
    L = load_library()
    cfg, classes, rates, lengths, prices, coeffs, tg = marshal(inp)
    per = (qsim_rep_stats * inp.R)() if per_rep else None
    tot = qsim_rep_stats()
    _check(L.qsim_simulate(C.byref(cfg), classes, _ptr(rates), _ptr(lengths), _ptr(prices), _ptr(coeffs), tg,
                           int(horizon_iters), C.byref(tot), per))
    out = _unpack(per, inp.R, inp.I) if per_rep else {}
    out["_totals"] = _unpack((tot,), 1, inp.I)
    return out


def simulate_waves(inp, horizon_iters: int, wave: int = 0) -> dict:
    """qsim_simulate_waves: all R replications of a whole run, `wave` of them resident at a time (0 = as many as fit)."""
    L = load_library()
    cfg, classes, rates, lengths, prices, coeffs, tg = marshal(inp)
    per = (qsim_rep_stats * inp.R)()
    tot = qsim_rep_stats()
    n = C.c_uint32()
    _check(L.qsim_simulate_waves(C.byref(cfg), classes, _ptr(rates), _ptr(lengths), _ptr(prices), _ptr(coeffs), tg,
                                 int(horizon_iters), int(wave), C.byref(tot), per, C.byref(n)))
    out = _unpack(per, inp.R, inp.I)
    out["_totals"] = _unpack((tot,), 1, inp.I)
    out["_waves"] = int(n.value)
    return out


def simulate_static(inp, horizon_iters: int, stream=None) -> dict:
    """qsim_simulate_static: like simulate_host, but the library allocates nothing; its state lives in a
    32 MiB array built into libqsim.so, so only small problems fit (a QSimError names the bytes needed).
    Meant for callers that may not call cudaMalloc; calls must not overlap on one GPU."""
    L = load_library()
    cfg, classes, rates, lengths, prices, coeffs, tg = marshal(inp)
    per = (qsim_rep_stats * inp.R)()
    tot = qsim_rep_stats()
    sp = C.c_void_p(stream.cuda_stream) if stream is not None else None
    _check(L.qsim_simulate_static(C.byref(cfg), classes, _ptr(rates), _ptr(lengths), _ptr(prices), _ptr(coeffs), tg,
                                  int(horizon_iters), C.byref(tot), per, sp))
    out = _unpack(per, inp.R, inp.I)
    out["_totals"] = _unpack((tot,), 1, inp.I)
    return out


class QSimCTMC:
    """The exponential-service model (qsim_ctmc_* of include/qsim.h) on a CtmcInputs; the workspace is a torch tensor."""

    def __init__(self, inp, device="cuda:0", stream=None):
        import torch
        if not torch.cuda.is_available():
            raise QSimError("no CUDA device: the simulator has no CPU path")
        self.L = load_library()
        self.inp = inp
        self.device = torch.device(device)
        self.cfg = qsim_ctmc_config(size=C.sizeof(qsim_ctmc_config), I=inp.I, N=inp.N, M=inp.M, B=inp.B, R=inp.R,
                                    qcap=inp.qcap, gate=inp.gate, router=inp.router, reserved=0, seed=inp.seed,
                                    rep_offset=inp.rep_offset)
        self.classes = (qsim_ctmc_class * inp.I)()
        for i in range(inp.I):
            self.classes[i] = qsim_ctmc_class(
                lam=float(inp.lam[i]), theta=float(inp.theta[i]), mu_p=float(inp.mu_p[i]), mu_m=float(inp.mu_m[i]),
                mu_s=float(inp.mu_s[i]), xstar=float(inp.xstar[i]), n_xstar=float(inp.n_xstar[i]),
                n_qpstar=float(inp.n_qpstar[i]), p_solo=float(inp.p_solo[i]), prio_rank=int(inp.prio_rank[i]), reserved=0)
        nbytes = C.c_size_t()
        _check(self.L.qsim_ctmc_workspace_bytes(C.byref(self.cfg), C.byref(nbytes)))
        self.nbytes = nbytes.value
        with torch.cuda.device(self.device):
            self.ws = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self.ptr = (self.ws.data_ptr() + 255) & ~255
            _check(self.L.qsim_ctmc_init(C.byref(self.cfg), self.classes, C.c_void_p(self.ptr), self.nbytes,
                                         C.c_void_p(self.stream.cuda_stream)))
        self.launches = 1

    def run_until(self, T_end: float) -> None:
        import torch
        n = C.c_uint64()
        with torch.cuda.device(self.device):
            _check(self.L.qsim_ctmc_run_until(C.byref(self.cfg), self.classes, C.c_void_p(self.ptr), self.nbytes,
                                              C.c_void_p(self.stream.cuda_stream), float(T_end), C.byref(n)))
        self.launches += n.value

    def stats(self) -> dict:
        import torch
        R, I = self.inp.R, self.inp.I
        per = (qsim_ctmc_rep_stats * R)()
        with torch.cuda.device(self.device):
            _check(self.L.qsim_ctmc_stats(C.byref(self.cfg), C.c_void_p(self.ptr), self.nbytes,
                                          C.c_void_p(self.stream.cuda_stream), per))
        raw = np.frombuffer(per, dtype=np.uint8).reshape(R, C.sizeof(qsim_ctmc_rep_stats))
        o_state = 10 * 8 * MAXI
        o_area = o_state + 5 * 4 * MAXI + 4 * MAXI
        cnt = raw[:, :o_state].copy().view(np.uint64).reshape(R, MAXI, 10)
        state = raw[:, o_state:o_state + 5 * 4 * MAXI].copy().view(np.uint32).reshape(R, MAXI, 5)
        area = raw[:, o_area:o_area + 5 * 8 * MAXI].copy().view(np.float64).reshape(R, MAXI, 5)
        tail = raw[:, o_area + 5 * 8 * MAXI:].copy()
        out = {}
        for k, n in enumerate(_CTMC_COUNTERS):
            out[n] = np.ascontiguousarray(cnt[:, :I, k])
        for k, n in enumerate(_STATE):
            out[n] = np.ascontiguousarray(state[:, :I, k])
        for k, n in enumerate(_CTMC_AREAS):
            out[n] = np.ascontiguousarray(area[:, :I, k])
        out["events"] = tail[:, :8].copy().view(np.uint64).reshape(R)
        out["T_elapsed"] = tail[:, 8:16].copy().view(np.float64).reshape(R)
        # per-GPU revenue rate of every replication under the instance's charging scheme (qsim_ctmc_revenue)
        rate = np.zeros(R, np.float64)
        P = np.ascontiguousarray(self.inp.P, np.float64); D = np.ascontiguousarray(self.inp.D, np.float64)
        prices = np.ascontiguousarray(self.inp.prices, np.float64)
        if (out["T_elapsed"] > 0).all():
            _check(self.L.qsim_ctmc_revenue(C.byref(self.cfg), per, _ptr(P), _ptr(D), _ptr(prices),
                                            1 if self.inp.meta.get("separate", False) else 0, _ptr(rate)))
        out["_revenue_rate"] = rate
        return out

    def close(self) -> None:
        self.ws = None
