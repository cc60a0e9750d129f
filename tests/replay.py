"""Independent re-derivation of a run from the oracle's event trace (pure Python, small cases only).

`Replay` walks the trace and rebuilds every queue, GPU and job from the logged events alone.  At each
step it checks the rules the paper states for any admissible policy and for gate-and-route:
capacity (Eq. (12)-(14)), FCFS and non-pre-emption (Section 2.3 "Admissible policies"), the gate's
argmin rule and the solo-first router (Section 4.1), token-by-token service (Section 2.2: one token per
active decode and one chunk of the prefill per iteration) and the iteration-time law (Eq. (1)-(3)).
It never calls the oracle's arithmetic; it only reads what the oracle logged.
"""
from __future__ import annotations

import math
from collections import defaultdict

EPS = 1e-12


class Replay:
    def __init__(self, inp, trace, rep=0):
        self.inp = inp
        self.tr = [e for e in trace if e["rep"] == rep]
        self.N, self.B, self.C, self.I = inp.N, inp.B, inp.C, inp.I
        self.blk = 0
        self.pq = [[] for _ in range(self.I)]          # waiting job ordinals per class (FCFS)
        self.dq = []                                   # (cls, job) finished prefill, waiting for a slot
        self.pf = [None] * self.N                      # (cls, job, remaining, t_admit)
        self.dec = [dict() for _ in range(self.N)]     # (cls, job) -> [tokens_left, t_place]
        self.iter_start = [None] * self.N              # start time of the running iteration
        self.batch = [None] * self.N                   # (p, d) frozen at iteration start
        self.X = [0] * self.I
        self.jobs = {}                                 # (cls, job) -> dict of timestamps and lengths
        self.sojourn = defaultdict(float)              # stage -> sum over jobs of time in stage (up to T)
        self.n_events = 0
        # (rank, size) of every choice the paper makes uniformly at random: the GPU inside the eligible tier
        # (Section 4.1) and the request that abandons a queue (memoryless patience, Section 2.3)
        self.place_ranks, self.admit_ranks, self.abandon_p_ranks, self.abandon_d_ranks = [], [], [], []
        self.max_load_seen = [0] * self.N              # most decodes ever held, per GPU

    # -- helpers -----------------------------------------------------------------------------
    def M(self):
        return int(self.inp.M[self.blk])

    def cap(self, g):
        return self.B - 1 if (g < self.M() or self.pf[g] is not None) else self.B

    def tau(self, p, d, K=0):
        """Eq. (1)-(3) plus the KV slope of the Section 6.1 solo fit: K = KV tokens resident in the batch."""
        am, beta, dm, a_s, ds, kappa = (float(x) for x in self.inp.coeffs)
        return (am + beta * p + dm * d if p > 0 else a_s + ds * d) + kappa * K

    def kv_tokens(self, g, members):
        """KV tokens held by the decodes of a batch: each one's prompt plus the tokens it has emitted so far."""
        K = 0
        for key in members:
            P, D = self.lengths(*key)
            K += P + (D - self.dec[g][key][0])
        return K

    def lengths(self, cls, job):
        j = self.jobs[(cls, job)]
        return j["P"], j["D"]

    def _maybe_start(self, g, t):
        """A GPU between iterations with work starts one at the current event time."""
        if self.iter_start[g] is None and (self.pf[g] is not None or self.dec[g]):
            p = min(self.C, self.pf[g][2]) if self.pf[g] is not None else 0
            self.iter_start[g] = t
            members = set(self.dec[g].keys())
            self.batch[g] = (p, len(members), members, self.kv_tokens(g, members))

    # -- the walk ----------------------------------------------------------------------------
    def run(self, known_lengths=None):
        """known_lengths: callable (cls, job) -> (P, D); defaults to the fixed class lengths."""
        inp = self.inp
        assert inp.router in (0, 3), "the replay models the single-buffer solo-first router and the no-router ablation"
        tr = self.tr
        k = 0
        while k < len(tr):
            t = tr[k]["t"]
            # one simulator event = the head record plus the decisions logged at the same time
            # before the next primary record
            group = [tr[k]]
            k += 1
            while k < len(tr) and tr[k]["type"] in ("ADMIT", "PLACE", "PREFILL_DONE", "DECODE_DONE", "OVERFLOW") \
                    and tr[k]["t"] == t:
                group.append(tr[k])
                k += 1
            self.n_events += 1
            touched = set()
            for e in group:
                typ, cls, g, job = e["type"], e["cls"], e["server"], e["job"]
                if typ == "BLOCK":
                    self.blk = job
                elif typ == "ARRIVAL":
                    P, D = known_lengths(cls, job) if known_lengths else (int(inp.P[cls]), int(inp.D[cls]))
                    self.jobs[(cls, job)] = dict(P=P, D=D, t_arr=t)
                    self.pq[cls].append(job)
                elif typ == "OVERFLOW":
                    if g < 0:
                        self.pq[cls].remove(job)
                        self.jobs[(cls, job)]["t_leave_q"] = t
                        self.jobs[(cls, job)]["dropped"] = True
                    else:
                        self.dq.remove((cls, job))
                        self.jobs[(cls, job)]["t_leave_dq"] = t
                        self.jobs[(cls, job)]["dropped"] = True
                elif typ == "ABANDON_P":
                    assert job in self.pq[cls]
                    self.abandon_p_ranks.append((self.pq[cls].index(job), len(self.pq[cls])))
                    self.pq[cls].remove(job)
                    self.jobs[(cls, job)]["t_leave_q"] = t
                elif typ == "ABANDON_D":
                    assert (cls, job) in self.dq
                    same = [e for e in self.dq if e[0] == cls]
                    self.abandon_d_ranks.append((same.index((cls, job)), len(same)))
                    self.dq.remove((cls, job))
                    self.jobs[(cls, job)]["t_leave_dq"] = t
                elif typ == "ITER_END":
                    self._iter_end(g, t, e["aux"], group)
                    touched.add(g)
                elif typ == "PREFILL_DONE":
                    pf = self.pf[g]
                    assert pf is not None and pf[0] == cls and pf[1] == job and pf[2] == 0, "prefill not finished"
                    self.pf[g] = None
                    self.X[cls] -= 1
                    self.jobs[(cls, job)]["t_pf"] = t
                    self.dq.append((cls, job))
                elif typ == "DECODE_DONE":
                    left, _ = self.dec[g][(cls, job)]
                    assert left == 0, "decode completed with tokens left"
                    del self.dec[g][(cls, job)]
                    self.jobs[(cls, job)]["t_done"] = t
                    self.jobs[(cls, job)]["g_dec"] = g
                elif typ == "PLACE":
                    self._check_place(cls, job, g, t)
                    touched.add(g)
                elif typ == "ADMIT":
                    self._check_admit(cls, job, g, t)
                    touched.add(g)
            # nothing may finish silently: every decode with 0 tokens left was logged as done
            for g in range(self.N):
                assert all(v[0] > 0 for v in self.dec[g].values()), "finished decode not completed"
                assert self.pf[g] is None or self.pf[g][2] > 0, "finished prefill not completed"
            self._check_work_conservation(t)
            for g in range(self.N):
                self._maybe_start(g, t)
        return self

    def _iter_end(self, g, t, tau_logged, group):
        assert self.iter_start[g] is not None, "iteration end on an idle GPU"
        p, d, members, K = self.batch[g]
        assert abs(tau_logged - self.tau(p, d, K)) < 1e-15, ("iteration time", tau_logged, self.tau(p, d, K), p, d, K)
        assert abs((self.iter_start[g] + tau_logged) - t) < 1e-9
        for key in members:                       # every decode frozen into the batch emits one token
            self.dec[g][key][0] -= 1
        if p > 0:
            c, j, rem, ta = self.pf[g]
            self.pf[g] = (c, j, rem - p, ta)
        self.iter_start[g] = None
        self.batch[g] = None

    def _check_place(self, cls, job, g, t):
        if self.inp.router == 3:
            # immediate same-slot decoding (EC ablation study): the request goes on where it prefilled, at once
            assert self.dq == [(cls, job)], "a request waited although there is no router"
            self.dq.pop()
            j = self.jobs[(cls, job)]
            assert g == j["g_pf"] and t == j["t_pf"], "decode must continue on the prefill GPU at prefill completion"
            assert self.pf[g] is None and len(self.dec[g]) < self.B, "more requests than slots on a GPU"
            self.dec[g][(cls, job)] = [self.lengths(cls, job)[1], t]
            j["t_place"] = t
            return
        # FCFS across classes in the single decode buffer
        assert self.dq and self.dq[0] == (cls, job), "decode buffer not FCFS"
        self.dq.pop(0)
        M = self.M()
        loads = [len(self.dec[h]) for h in range(self.N)]
        assert loads[g] < self.cap(g), "decode cap exceeded (Eq. (13)-(14))"
        solo_free = [h for h in range(M, self.N) if loads[h] < self.cap(h)]
        mix_free = [h for h in range(0, M) if loads[h] < self.cap(h)]
        tier = solo_free if solo_free else mix_free
        assert g in tier, "router must fill solo GPUs first (Section 4.1)"
        self.place_ranks.append((tier.index(g), len(tier)))
        if self.inp.placement == 1:
            best = min(tier, key=lambda h: (loads[h], h))
            assert g == best, "least-loaded placement violated"
        P, D = self.lengths(cls, job)
        self.dec[g][(cls, job)] = [D, t]
        self.max_load_seen[g] = max(self.max_load_seen[g], len(self.dec[g]))
        self.jobs[(cls, job)]["t_place"] = t

    def _check_admit(self, cls, job, g, t):
        inp = self.inp
        M = self.M()
        assert g < M, "prefill on a solo GPU"
        assert self.pf[g] is None, "two prefills on one GPU (Eq. (12))"
        assert self.pq[cls] and self.pq[cls][0] == job, "prefill queue not FCFS within class"
        waiting = [i for i in range(self.I) if self.pq[i]]
        if inp.gate == 0:
            xs, nx, nq = inp.xstar[self.blk], inp.n_xstar[self.blk], inp.n_qpstar[self.blk]
            cand = [i for i in waiting if xs[i] > 0]
            key = {i: ((self.X[i] - nx[i]) / xs[i], -(len(self.pq[i]) - nq[i]), i) for i in cand}
            assert cls == min(cand, key=lambda i: key[i]), ("occupancy gate argmin violated", key, cls)
        elif inp.gate == 2:
            oldest = min(waiting, key=lambda i: (self.jobs[(i, self.pq[i][0])]["t_arr"], i))
            assert cls == oldest, "FCFS gate violated"
        else:
            assert cls == min(waiting, key=lambda i: (int(inp.prio_rank[i]), i)), "priority gate violated"
        cands = [h for h in range(M) if self.pf[h] is None and len(self.dec[h]) <= self.B - 1]
        assert g in cands
        self.admit_ranks.append((cands.index(g), len(cands)))
        if inp.placement == 1:
            assert g == min(cands, key=lambda h: (len(self.dec[h]), h))
        self.pq[cls].pop(0)
        P, D = self.lengths(cls, job)
        self.pf[g] = (cls, job, P, t)
        self.X[cls] += 1
        self.jobs[(cls, job)]["t_admit"] = t
        self.jobs[(cls, job)]["g_pf"] = g

    def _check_work_conservation(self, t):
        """After an event's decisions nothing placeable is left waiting."""
        M = self.M()
        if self.dq:
            free = [h for h in range(self.N) if len(self.dec[h]) < self.cap(h)]
            assert not free, "decode buffer non-empty while a slot is free"
        idle = [h for h in range(M) if self.pf[h] is None and len(self.dec[h]) <= self.B - 1]
        if idle:
            if self.inp.gate == 0:
                waiting = [i for i in range(self.I) if self.pq[i] and self.inp.xstar[self.blk][i] > 0]
            else:
                waiting = [i for i in range(self.I) if self.pq[i]]
            assert not waiting, "idle prefill slot while an admissible class waits"

    # -- Little identity -----------------------------------------------------------------------
    def stage_time(self, T):
        """Sum over jobs of the time spent in each stage up to T, per class."""
        out = {s: [0.0] * self.I for s in ("Qp", "X", "Qd", "Y")}
        for (cls, _), j in self.jobs.items():
            t_in = j["t_arr"]
            t_out = j.get("t_admit", j.get("t_leave_q", T))
            out["Qp"][cls] += min(T, t_out) - t_in
            if "t_admit" in j:
                out["X"][cls] += min(T, j.get("t_pf", T)) - j["t_admit"]
            if "t_pf" in j:
                out["Qd"][cls] += min(T, j.get("t_place", j.get("t_leave_dq", T))) - j["t_pf"]
            if "t_place" in j:
                out["Y"][cls] += min(T, j.get("t_done", T)) - j["t_place"]
        return out


def expected_counts(rp: Replay):
    """Per-class counters re-derived from the replayed job table."""
    I = rp.I
    c = {k: [0] * I for k in ("arrivals", "admitted", "prefill_done", "placed", "done", "abandoned_p", "abandoned_d")}
    for (cls, _), j in rp.jobs.items():
        c["arrivals"][cls] += 1
        c["admitted"][cls] += "t_admit" in j
        c["prefill_done"][cls] += "t_pf" in j
        c["placed"][cls] += "t_place" in j
        c["done"][cls] += "t_done" in j
        c["abandoned_p"][cls] += "t_leave_q" in j and not j.get("dropped")
        c["abandoned_d"][cls] += "t_leave_dq" in j and not j.get("dropped")
    return c


def isclose(a, b, rel=1e-9):
    return math.isclose(a, b, rel_tol=rel, abs_tol=1e-9)
