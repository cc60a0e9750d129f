// Exponential-service model of the gate-and-route network (Section 2.3): device kernel and C ABI.
// Included at the end of qsim_lib.cu (it uses that file's error helpers and the Philox / qlog routines of
// qsim_device.cuh).
//
// Requests of a class are exchangeable here, so a replication is a handful of integers per class plus the
// class order of its decode buffers: one THREAD simulates one replication, and a warp advances 32
// replications at once.  Every class has seven unit-rate Poisson processes (arrivals, abandonment from the
// prefill queue, abandonment from each decode buffer, prefill completions, mixed and solo decode
// completions) that run on the integrated intensities of Eq. (7)-(9): a process with intensity c n(t) keeps
// the integral acc of c n since its last jump and the exponential level lvl of its next jump, and its jump
// time is recomputed whenever n changes.  Per event a thread scans its 7 I jump times, applies the jump,
// lets the policy act (decode buffers into free slots, solo group first; then the prefill gate) and updates
// the clocks whose counts changed.  All clock arithmetic is single IEEE operations in a fixed order.
// While a launch runs, a replication's clocks, counts and statistics sit in shared memory (word w of thread t
// at w * blockDim + t); the four processes that take one request out of one count share one code path, so
// the threads of a warp diverge only between arrivals, buffer abandonments and that path.
#pragma once

namespace qsimdev {

enum { CK_ARR = 0, CK_ABP = 1, CK_ABD0 = 2, CK_ABD1 = 3, CK_SP = 4, CK_SDM = 5, CK_SDS = 6, CK_N = 7 };
enum { CC_ARRIVALS = 0, CC_ADMITTED, CC_PREFILL_DONE, CC_PLACED_MIXED, CC_PLACED_SOLO, CC_DONE_MIXED, CC_DONE_SOLO,
       CC_ABANDONED_P, CC_ABANDONED_D, CC_OVERFLOW_D, CC_N };
enum { CA_QP = 0, CA_X, CA_QD, CA_YM, CA_YS, CA_N };

struct CtmcClk { double acc, lvl, t_last, t_fire; unsigned long long m; };

// state of one replication in global memory between launches
struct CtmcRep {
    double T_end;
    unsigned long long events;
    uint32_t head[2], n[2];
    uint32_t err, done;
    CtmcClk clk[CK_N][MAXI];
    uint32_t Qp[MAXI], X[MAXI], Qd[2][MAXI], Ym[MAXI], Ys[MAXI];
    unsigned long long sli_ord[MAXI];
    double area[CA_N][MAXI], area_t[CA_N][MAXI];
    unsigned long long cnt[MAXI][CC_N];
};

struct CtmcClassPar { double lambda, theta, mu_p, mu_m, mu_s, xstar, nx, nq, ps; uint32_t prio, pad; };

struct CtmcParams {
    uint32_t I, N, M, B, R, qcap, gate, router, init, pad;
    unsigned long long seed, rep_offset, event_budget;
    double T_end;
    CtmcClassPar cls[MAXI];
    CtmcRep *reps;          // [R]
    uint8_t *rings;         // [R][2][qcap] class ids of the decode buffers, FCFS
    uint32_t *not_done;
};

// Working copy of one replication in shared memory: 8-byte words, word w of thread t at [w * blockDim + t]
// (consecutive threads hit consecutive banks).  Only the I classes in use take space: 5 + 47 I words.  The event
// counters and the time integrals are only ever added to, so they stay in the global record and take
// fire-and-forget additions (one thread, one address: applied in program order, so the sums are deterministic).
struct CtmcWords {
    unsigned long long *base;   // this thread's word 0
    uint32_t stride, I;
    enum { W_EVENTS = 0, W_HEAD0 = 1, W_HEAD1 = 2, W_N0 = 3, W_N1 = 4, W_BASE = 5 };
    __device__ __forceinline__ uint32_t clk(uint32_t k, uint32_t i, uint32_t f) const { return W_BASE + (k * I + i) * 5u + f; }   // f: acc, lvl, t_last, t_fire, m
    __device__ __forceinline__ uint32_t count(uint32_t c, uint32_t i) const { return W_BASE + 35u * I + c * I + i; }             // c: Qp, X, Qd0, Qd1, Ym, Ys
    __device__ __forceinline__ uint32_t sli(uint32_t i) const { return W_BASE + 41u * I + i; }
    __device__ __forceinline__ uint32_t area_t(uint32_t a, uint32_t i) const { return W_BASE + 42u * I + a * I + i; }
    __host__ __device__ static uint32_t words(uint32_t I) { return 5u + 47u * I; }
    __device__ __forceinline__ unsigned long long u(uint32_t w) const { return base[(size_t)w * stride]; }
    __device__ __forceinline__ void su(uint32_t w, unsigned long long v) const { base[(size_t)w * stride] = v; }
    __device__ __forceinline__ double d(uint32_t w) const { return __longlong_as_double((long long)u(w)); }
    __device__ __forceinline__ void sd(uint32_t w, double v) const { su(w, (unsigned long long)__double_as_longlong(v)); }
};
enum { CQ_QP = 0, CQ_X = 1, CQ_QD0 = 2, CQ_QD1 = 3, CQ_YM = 4, CQ_YS = 5 };

struct CtmcSim {
    const CtmcParams &p;
    const CtmcWords W;
    CtmcRep &G;                 // the record in global memory: counters and integrals are added to in place
    uint8_t *ring0, *ring1;
    const uint32_t rep;
    uint32_t totX, totYm, totYs, err;

    __device__ CtmcSim(const CtmcParams &p_, const CtmcWords &W_, CtmcRep &G_, uint32_t rep_)
        : p(p_), W(W_), G(G_), ring0(p_.rings + (size_t)rep_ * 2 * p_.qcap), ring1(ring0 + p_.qcap), rep(rep_), totX(0), totYm(0), totYs(0), err(0) {}

    __device__ __forceinline__ uint32_t stream_of(uint32_t k, uint32_t i) const
    {
        const uint32_t purpose = k < CK_SP ? k : k + 4u;      // 0..3 as in the iteration-level simulator, then 8, 9, 10
        return (purpose << 8) | i;
    }
    __device__ __forceinline__ void rnd(uint32_t stream, unsigned long long index, uint32_t &w0, uint32_t &w1, uint32_t &w2, uint32_t &w3) const
    {
        const unsigned long long grep = p.rep_offset + rep;
        philox((uint32_t)index, (uint32_t)(index >> 32), stream, (uint32_t)grep, (uint32_t)p.seed, (uint32_t)(p.seed >> 32), w0, w1, w2, w3);
    }
    // intensity of process k of class i per unit of the count it runs on (the arrival process runs on the constant 1)
    __device__ __forceinline__ double coef(uint32_t k, uint32_t i) const
    {
        const CtmcClassPar &c = p.cls[i];
        return k <= CK_ABD1 ? (k == CK_ARR ? __dmul_rn((double)p.N, c.lambda) : c.theta)
                            : (k == CK_SP ? c.mu_p : (k == CK_SDM ? c.mu_m : c.mu_s));
    }
    __device__ __forceinline__ uint32_t cq(uint32_t c, uint32_t i) const { return (uint32_t)W.u(W.count(c, i)); }
    __device__ __forceinline__ void touch(uint32_t a, uint32_t i, uint32_t count, double t)
    {
        atomicAdd(&G.area[a][i], __dmul_rn((double)count, __dsub_rn(t, W.d(W.area_t(a, i)))));
        W.sd(W.area_t(a, i), t);
    }
    // the count that process k of class i runs on changes from n_old to n_new at time t
    __device__ void clk_change(uint32_t k, uint32_t i, uint32_t n_old, uint32_t n_new, double t)
    {
        const double c = coef(k, i);
        if (!(c > 0.0)) return;
        const double acc = __dadd_rn(W.d(W.clk(k, i, 0)), __dmul_rn(__dmul_rn(c, (double)n_old), __dsub_rn(t, W.d(W.clk(k, i, 2)))));
        W.sd(W.clk(k, i, 0), acc);
        W.sd(W.clk(k, i, 2), t);
        double tf = dinf();
        if (n_new > 0) {
            double rem = __dsub_rn(W.d(W.clk(k, i, 1)), acc);
            if (rem < 0.0) rem = 0.0;
            tf = __dadd_rn(t, __ddiv_rn(rem, __dmul_rn(c, (double)n_new)));
        }
        W.sd(W.clk(k, i, 3), tf);
    }
    // process k of class i has just jumped at t and its count is now n_new: next level from draw m
    __device__ void clk_fired(uint32_t k, uint32_t i, uint32_t n_new, double t, uint32_t &w2)
    {
        const unsigned long long m = W.u(W.clk(k, i, 4));
        uint32_t w0, w1, w3;
        rnd(stream_of(k, i), m, w0, w1, w2, w3);
        const double lvl = -qlog(u53(w0, w1));
        W.sd(W.clk(k, i, 1), lvl);
        W.su(W.clk(k, i, 4), m + 1);
        W.sd(W.clk(k, i, 0), 0.0);
        W.sd(W.clk(k, i, 2), t);
        W.sd(W.clk(k, i, 3), n_new > 0 ? __dadd_rn(t, __ddiv_rn(lvl, __dmul_rn(coef(k, i), (double)n_new))) : dinf());
    }
    // setters that keep the time integral and the process that runs on the count in step
    __device__ void set_count(uint32_t c, uint32_t i, uint32_t v, double t)
    {
        // c -> (process, integral): Qp -> (ABP, Q_p), X -> (SP, X), Ym -> (SDM, Y_m), Ys -> (SDS, Y_s)
        const uint32_t k = c == CQ_QP ? CK_ABP : (c == CQ_X ? CK_SP : (c == CQ_YM ? CK_SDM : CK_SDS));
        const uint32_t a = c == CQ_QP ? CA_QP : (c == CQ_X ? CA_X : (c == CQ_YM ? CA_YM : CA_YS));
        const uint32_t old = cq(c, i);
        clk_change(k, i, old, v, t);
        touch(a, i, old, t);
        W.su(W.count(c, i), v);
        if (c == CQ_X) totX += v - old;
        if (c == CQ_YM) totYm += v - old;
        if (c == CQ_YS) totYs += v - old;
    }
    __device__ void set_Qd(uint32_t pool, uint32_t i, uint32_t v, double t)
    {
        const uint32_t q0 = cq(CQ_QD0, i), q1 = cq(CQ_QD1, i);
        clk_change(pool ? CK_ABD1 : CK_ABD0, i, pool ? q1 : q0, v, t);
        touch(CA_QD, i, q0 + q1, t);
        W.su(W.count(pool ? CQ_QD1 : CQ_QD0, i), v);
    }
    __device__ __forceinline__ void bump(uint32_t i, uint32_t c) { atomicAdd(&G.cnt[i][c], 1ull); }

    // Section 4.1 occupancy gate (xi_i = (X_i - n x*_i)/x*_i, ties to the largest Q_p,i - n q*_p,i) or the
    // Section 5.1.1 priority gate (smallest static rank); ties to the lowest class index
    __device__ uint32_t gate_class() const
    {
        uint32_t best = NONE32;
        if (p.gate == 1) {
            for (uint32_t i = 0; i < p.I; ++i)
                if (cq(CQ_QP, i) > 0 && (best == NONE32 || p.cls[i].prio < p.cls[best].prio)) best = i;
            return best;
        }
        double bxi = 0.0, bdq = 0.0;
        for (uint32_t i = 0; i < p.I; ++i) {
            const uint32_t Qp = cq(CQ_QP, i);
            if (Qp == 0 || !(p.cls[i].xstar > 0.0)) continue;
            const double xi = __ddiv_rn(__dsub_rn((double)cq(CQ_X, i), p.cls[i].nx), p.cls[i].xstar);
            const double dq = __dsub_rn((double)Qp, p.cls[i].nq);
            if (best == NONE32 || xi < bxi || (xi == bxi && dq > bdq)) { best = i; bxi = xi; bdq = dq; }
        }
        return best;
    }

    __device__ void dispatch(double t)
    {
        const uint32_t cap_s = (p.N - p.M) * p.B, cap_m = p.M * (p.B - 1u);
        const uint32_t npools = p.router == 1 ? 2u : 1u;
        for (uint32_t pool = 0; pool < npools; ++pool) {
            uint8_t *ring = pool ? ring1 : ring0;
            const uint32_t wn = pool ? CtmcWords::W_N1 : CtmcWords::W_N0, wh = pool ? CtmcWords::W_HEAD1 : CtmcWords::W_HEAD0;
            uint32_t n = (uint32_t)W.u(wn);
            while (n > 0) {
                bool to_solo;
                if (p.router == 1) {
                    to_solo = pool == 0;
                    if (to_solo ? totYs >= cap_s : totYm >= cap_m) break;
                } else {
                    if (totYs < cap_s) to_solo = true;
                    else if (totYm < cap_m) to_solo = false;
                    else break;
                }
                uint32_t head = (uint32_t)W.u(wh);
                const uint32_t i = ring[head];
                head = head + 1 == p.qcap ? 0 : head + 1;
                W.su(wh, head);
                n -= 1;
                W.su(wn, n);
                set_Qd(pool, i, cq(pool ? CQ_QD1 : CQ_QD0, i) - 1, t);
                set_count(to_solo ? CQ_YS : CQ_YM, i, cq(to_solo ? CQ_YS : CQ_YM, i) + 1, t);
                bump(i, to_solo ? CC_PLACED_SOLO : CC_PLACED_MIXED);
            }
        }
        while (totX < p.M) {
            const uint32_t i = gate_class();
            if (i == NONE32) break;
            set_count(CQ_QP, i, cq(CQ_QP, i) - 1, t);
            set_count(CQ_X, i, cq(CQ_X, i) + 1, t);
            bump(i, CC_ADMITTED);
        }
    }

    // empty system at t = 0: every process gets its first level, the arrival processes their first jump time
    __device__ void init()
    {
        for (uint32_t w = 0; w < CtmcWords::words(p.I); ++w) W.su(w, 0ull);
        for (uint32_t i = 0; i < p.I; ++i) {
            for (uint32_t k = 0; k < CK_N; ++k) {
                uint32_t w0, w1, w2, w3;
                rnd(stream_of(k, i), 0, w0, w1, w2, w3);
                W.sd(W.clk(k, i, 1), -qlog(u53(w0, w1)));
                W.sd(W.clk(k, i, 3), dinf());
                W.su(W.clk(k, i, 4), 1ull);
            }
            const double Lam = __dmul_rn((double)p.N, p.cls[i].lambda);
            if (Lam > 0.0) W.sd(W.clk(CK_ARR, i, 3), __dadd_rn(0.0, __ddiv_rn(W.d(W.clk(CK_ARR, i, 1)), Lam)));
        }
    }

    // events with t <= T_end, at most `budget` of them; returns true when none is left up to T_end
    __device__ bool run(double T_end, unsigned long long budget)
    {
        for (uint32_t i = 0; i < p.I; ++i) { totX += cq(CQ_X, i); totYm += cq(CQ_YM, i); totYs += cq(CQ_YS, i); }
        unsigned long long events = W.u(CtmcWords::W_EVENTS);
        bool finished;
        for (;;) {
            // earliest process; ties by process kind, then class (strict '<' in that scan order)
            double te = dinf();
            uint32_t bk = 0, bi = 0;
#pragma unroll
            for (uint32_t k = 0; k < CK_N; ++k)
                for (uint32_t i = 0; i < p.I; ++i) {
                    const double tf = W.d(W.clk(k, i, 3));
                    if (tf < te) { te = tf; bk = k; bi = i; }
                }
            if (!(te <= T_end)) { finished = true; break; }
            if (budget == 0) { finished = false; break; }
            --budget;
            const double t = te;
            const uint32_t i = bi;
            ++events;
            uint32_t w2 = 0;
            if (bk == CK_ABD0 || bk == CK_ABD1) {
                const uint32_t pool = bk == CK_ABD1 ? 1u : 0u;
                const uint32_t Q = cq(pool ? CQ_QD1 : CQ_QD0, i);
                clk_fired(bk, i, Q - 1, t, w2);
                // a uniformly chosen waiting class-i request leaves the pool's buffer; the rest keep their order
                uint8_t *ring = pool ? ring1 : ring0;
                const uint32_t wn = pool ? CtmcWords::W_N1 : CtmcWords::W_N0;
                uint32_t rank = __umulhi(w2, Q), pos = 0;
                const uint32_t n = (uint32_t)W.u(wn), head = (uint32_t)W.u(pool ? CtmcWords::W_HEAD1 : CtmcWords::W_HEAD0);
                for (pos = 0; pos < n; ++pos) {
                    uint32_t a = head + pos; if (a >= p.qcap) a -= p.qcap;
                    if (ring[a] != i) continue;
                    if (rank == 0) break;
                    --rank;
                }
                if (pos >= n) { err = ERR_INTERNAL; finished = true; break; }
                for (uint32_t k = pos; k + 1 < n; ++k) {
                    uint32_t a = head + k, b = head + k + 1;
                    if (a >= p.qcap) a -= p.qcap;
                    if (b >= p.qcap) b -= p.qcap;
                    ring[a] = ring[b];
                }
                W.su(wn, n - 1);
                touch(CA_QD, i, cq(CQ_QD0, i) + cq(CQ_QD1, i), t);
                W.su(W.count(pool ? CQ_QD1 : CQ_QD0, i), Q - 1);
                bump(i, CC_ABANDONED_D);
            } else {
                // One code path for the five processes that move one request across one count: an arrival adds one to the
                // prefill queue (and redraws on the constant count 1); abandonment from the prefill queue, prefill
                // completion and mixed / solo decode completion take one out of the count they run on.
                const bool arr = bk == CK_ARR;
                const uint32_t c = (arr || bk == CK_ABP) ? CQ_QP : (bk == CK_SP ? CQ_X : (bk == CK_SDM ? CQ_YM : CQ_YS));
                const uint32_t a = (arr || bk == CK_ABP) ? CA_QP : (bk == CK_SP ? CA_X : (bk == CK_SDM ? CA_YM : CA_YS));
                const uint32_t cc = arr ? CC_ARRIVALS : (bk == CK_ABP ? CC_ABANDONED_P : (bk == CK_SP ? CC_PREFILL_DONE : (bk == CK_SDM ? CC_DONE_MIXED : CC_DONE_SOLO)));
                const uint32_t old = cq(c, i), now = arr ? old + 1 : old - 1;
                if (arr) clk_change(CK_ABP, i, old, now, t);       // the queue's abandonment process sees the new length
                touch(a, i, old, t);
                W.su(W.count(c, i), now);
                totX -= bk == CK_SP ? 1u : 0u; totYm -= bk == CK_SDM ? 1u : 0u; totYs -= bk == CK_SDS ? 1u : 0u;
                bump(i, cc);
                clk_fired(bk, i, arr ? 1u : now, t, w2);
                if (bk == CK_SP) {
                    uint32_t pool = 0;
                    if (p.router == 1) {
                        // SLI-aware router: one uniform per finished prefill decides the pool (Section 5.2)
                        const unsigned long long ord = W.u(W.sli(i));
                        W.su(W.sli(i), ord + 1);
                        uint32_t w0, w1, w3;
                        rnd((STREAM_SLI << 8) | i, ord, w0, w1, w2, w3);
                        pool = u53(w0, w1) <= p.cls[i].ps ? 0u : 1u;
                    }
                    const uint32_t wn = pool ? CtmcWords::W_N1 : CtmcWords::W_N0;
                    const uint32_t n = (uint32_t)W.u(wn);
                    if (n >= p.qcap) {
                        bump(i, CC_OVERFLOW_D);
                    } else {
                        uint32_t pos = (uint32_t)W.u(pool ? CtmcWords::W_HEAD1 : CtmcWords::W_HEAD0) + n; if (pos >= p.qcap) pos -= p.qcap;
                        (pool ? ring1 : ring0)[pos] = (uint8_t)i;
                        W.su(wn, n + 1);
                        set_Qd(pool, i, cq(pool ? CQ_QD1 : CQ_QD0, i) + 1, t);
                    }
                }
            }
            dispatch(t);
        }
        W.su(CtmcWords::W_EVENTS, events);
        return finished;
    }

    // the record in global memory <-> the working copy
    __device__ void load(const CtmcRep &S)
    {
        W.su(CtmcWords::W_EVENTS, S.events);
        W.su(CtmcWords::W_HEAD0, S.head[0]); W.su(CtmcWords::W_HEAD1, S.head[1]); W.su(CtmcWords::W_N0, S.n[0]); W.su(CtmcWords::W_N1, S.n[1]);
        for (uint32_t i = 0; i < p.I; ++i) {
            for (uint32_t k = 0; k < CK_N; ++k) {
                const CtmcClk &q = S.clk[k][i];
                W.sd(W.clk(k, i, 0), q.acc); W.sd(W.clk(k, i, 1), q.lvl); W.sd(W.clk(k, i, 2), q.t_last); W.sd(W.clk(k, i, 3), q.t_fire);
                W.su(W.clk(k, i, 4), q.m);
            }
            W.su(W.count(CQ_QP, i), S.Qp[i]); W.su(W.count(CQ_X, i), S.X[i]); W.su(W.count(CQ_QD0, i), S.Qd[0][i]);
            W.su(W.count(CQ_QD1, i), S.Qd[1][i]); W.su(W.count(CQ_YM, i), S.Ym[i]); W.su(W.count(CQ_YS, i), S.Ys[i]);
            W.su(W.sli(i), S.sli_ord[i]);
            for (uint32_t a = 0; a < CA_N; ++a) W.sd(W.area_t(a, i), S.area_t[a][i]);
        }
    }
    __device__ void store(CtmcRep &S) const
    {
        S.events = W.u(CtmcWords::W_EVENTS);
        S.head[0] = (uint32_t)W.u(CtmcWords::W_HEAD0); S.head[1] = (uint32_t)W.u(CtmcWords::W_HEAD1);
        S.n[0] = (uint32_t)W.u(CtmcWords::W_N0); S.n[1] = (uint32_t)W.u(CtmcWords::W_N1);
        for (uint32_t i = 0; i < p.I; ++i) {
            for (uint32_t k = 0; k < CK_N; ++k) {
                CtmcClk &q = S.clk[k][i];
                q.acc = W.d(W.clk(k, i, 0)); q.lvl = W.d(W.clk(k, i, 1)); q.t_last = W.d(W.clk(k, i, 2)); q.t_fire = W.d(W.clk(k, i, 3));
                q.m = W.u(W.clk(k, i, 4));
            }
            S.Qp[i] = cq(CQ_QP, i); S.X[i] = cq(CQ_X, i); S.Qd[0][i] = cq(CQ_QD0, i); S.Qd[1][i] = cq(CQ_QD1, i);
            S.Ym[i] = cq(CQ_YM, i); S.Ys[i] = cq(CQ_YS, i);
            S.sli_ord[i] = W.u(W.sli(i));
            for (uint32_t a = 0; a < CA_N; ++a) S.area_t[a][i] = W.d(W.area_t(a, i));
        }
    }
};

// One thread per replication.  The replication's record lives in global memory between launches; a launch works on a
// copy in shared memory.  init != 0: start from the empty system at t = 0 (no events are processed).
__global__ void __launch_bounds__(64) qsim_ctmc_kernel(CtmcParams p)
{
    extern __shared__ __align__(16) unsigned long long ctmc_sm[];
    const uint32_t rep = blockIdx.x * blockDim.x + threadIdx.x;
    if (rep >= p.R) return;
    CtmcRep &S = p.reps[rep];
    CtmcWords W;
    W.base = ctmc_sm + threadIdx.x; W.stride = blockDim.x; W.I = p.I;
    CtmcSim sim(p, W, S, rep);
    if (p.init) {
        uint32_t *w = reinterpret_cast<uint32_t *>(&S);
        for (uint32_t o = 0; o < sizeof(CtmcRep) / 4; ++o) w[o] = 0;
        sim.init();
        sim.store(S);
        S.done = 1;
        return;
    }
    if (S.err || (S.done && S.T_end == p.T_end)) return;
    sim.load(S);
    const bool finished = sim.run(p.T_end, p.event_budget);
    sim.store(S);
    S.T_end = p.T_end;
    S.err = sim.err;
    S.done = finished ? 1u : 0u;
    if (!finished) atomicAdd(p.not_done, 1u);
}

}  // namespace qsimdev

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------
namespace {

int ctmc_validate(const qsim_ctmc_config *cfg, const qsim_ctmc_class *cls)
{
    if (!cfg || !cls) return fail(QSIM_EINVAL, "null argument");
    if (cfg->size != sizeof(qsim_ctmc_config)) return fail(QSIM_EINVAL, "qsim_ctmc_config.size does not match this library");
    if (cfg->I < 1 || cfg->I > QSIM_MAXI || cfg->N < 1 || cfg->M > cfg->N || cfg->B < 1 || cfg->R < 1 || cfg->qcap < 1)
        return fail(QSIM_EINVAL, "need 1 <= I <= 8, N >= 1, M <= N, B >= 1, R >= 1, qcap >= 1");
    if ((uint64_t)cfg->N * cfg->B > 0x7fffffffull) return fail(QSIM_EINVAL, "N * B too large");
    if (cfg->gate > QSIM_GATE_PRIORITY || cfg->router > QSIM_ROUTER_SLI)
        return fail(QSIM_EINVAL, "the exponential-service model has the occupancy and priority gates and the solo-first and SLI routers");
    for (uint32_t i = 0; i < cfg->I; ++i) {
        const qsim_ctmc_class &c = cls[i];
        const double v[9] = { c.lambda, c.theta, c.mu_p, c.mu_m, c.mu_s, c.xstar, c.n_xstar, c.n_qpstar, c.p_solo };
        for (double x : v)
            if (!std::isfinite(x) || x < 0.0) return fail(QSIM_EINVAL, "class parameters must be finite and non-negative");
        if (!(c.mu_p > 0.0) || !(c.mu_m > 0.0) || !(c.mu_s > 0.0)) return fail(QSIM_EINVAL, "service rates must be positive");
        if (c.p_solo > 1.0) return fail(QSIM_EINVAL, "p_solo must lie in [0, 1]");
    }
    return QSIM_OK;
}

struct CtmcSections { size_t reps, rings, flag, total; };

CtmcSections ctmc_sections(const qsim_ctmc_config &c)
{
    CtmcSections s;
    size_t o = 0;
    s.reps = o; o = align256(o + (size_t)c.R * sizeof(CtmcRep));
    s.rings = o; o = align256(o + (size_t)c.R * 2 * c.qcap);
    s.flag = o; o = align256(o + 4);
    s.total = o;
    return s;
}

// one warp per block: many small blocks spread the replications over all SMs; the working copies of a block's
// replications take 32 (5 + 47 I) 8-byte words of shared memory
int ctmc_launch_shape(uint32_t I, uint32_t &threads, size_t &smem)
{
    threads = 32;
    smem = (size_t)threads * CtmcWords::words(I) * 8;
    if (smem > 48u * 1024u)
        CUDA_TRY(cudaFuncSetAttribute(qsim_ctmc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return QSIM_OK;
}

int ctmc_params(const qsim_ctmc_config *cfg, const qsim_ctmc_class *cls, void *ws, size_t bytes, CtmcParams &p)
{
    int rc = ctmc_validate(cfg, cls);
    if (rc != QSIM_OK) return rc;
    const CtmcSections sec = ctmc_sections(*cfg);
    if (!ws) return fail(QSIM_EWORKSPACE, "workspace pointer is null");
    if (bytes < sec.total) return fail(QSIM_EWORKSPACE, "workspace too small: need " + std::to_string(sec.total) + " bytes");
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return fail(QSIM_EWORKSPACE, "workspace must be 256-byte aligned");
    std::memset(&p, 0, sizeof p);
    p.I = cfg->I; p.N = cfg->N; p.M = cfg->M; p.B = cfg->B; p.R = cfg->R; p.qcap = cfg->qcap; p.gate = cfg->gate; p.router = cfg->router;
    p.seed = cfg->seed; p.rep_offset = cfg->rep_offset; p.event_budget = 1ull << 26;
    for (uint32_t i = 0; i < cfg->I; ++i) {
        CtmcClassPar &c = p.cls[i];
        c.lambda = cls[i].lambda; c.theta = cls[i].theta; c.mu_p = cls[i].mu_p; c.mu_m = cls[i].mu_m; c.mu_s = cls[i].mu_s;
        c.xstar = cls[i].xstar; c.nx = cls[i].n_xstar; c.nq = cls[i].n_qpstar; c.ps = cls[i].p_solo; c.prio = cls[i].prio_rank;
    }
    char *base = static_cast<char *>(ws);
    p.reps = reinterpret_cast<CtmcRep *>(base + sec.reps);
    p.rings = reinterpret_cast<uint8_t *>(base + sec.rings);
    p.not_done = reinterpret_cast<uint32_t *>(base + sec.flag);
    return QSIM_OK;
}

}  // namespace

extern "C" {

int qsim_ctmc_workspace_bytes(const qsim_ctmc_config *cfg, size_t *bytes)
{
    if (!cfg || !bytes) return fail(QSIM_EINVAL, "null argument");
    if (cfg->size != sizeof(qsim_ctmc_config) || cfg->R < 1 || cfg->qcap < 1) return fail(QSIM_EINVAL, "bad qsim_ctmc_config");
    *bytes = ctmc_sections(*cfg).total;
    return QSIM_OK;
}

int qsim_ctmc_init(const qsim_ctmc_config *cfg, const qsim_ctmc_class *classes, void *dev_workspace, size_t bytes, void *cuda_stream)
{
    CtmcParams p;
    int rc = ctmc_params(cfg, classes, dev_workspace, bytes, p);
    if (rc != QSIM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    p.init = 1;
    uint32_t threads = 0;
    size_t smem = 0;
    rc = ctmc_launch_shape(cfg->I, threads, smem);
    if (rc != QSIM_OK) return rc;
    qsim_ctmc_kernel<<<(cfg->R + threads - 1u) / threads, threads, smem, st>>>(p);
    CUDA_TRY(cudaGetLastError());
    return QSIM_OK;
}

int qsim_ctmc_run_until(const qsim_ctmc_config *cfg, const qsim_ctmc_class *classes, void *dev_workspace, size_t bytes,
                        void *cuda_stream, double T_end, uint64_t *launches)
{
    CtmcParams p;
    int rc = ctmc_params(cfg, classes, dev_workspace, bytes, p);
    if (rc != QSIM_OK) return rc;
    if (!(T_end >= 0.0) || !std::isfinite(T_end)) return fail(QSIM_EINVAL, "T_end must be finite and non-negative");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    p.T_end = T_end;
    uint64_t n = 0;
    uint32_t threads = 0;
    size_t smem = 0;
    rc = ctmc_launch_shape(cfg->I, threads, smem);
    if (rc != QSIM_OK) return rc;
    // a replication that used up its per-launch event budget is continued by further launches
    uint32_t flag = 1;
    for (int guard = 0; guard < 100000 && flag != 0; ++guard) {
        CUDA_TRY(cudaMemsetAsync(p.not_done, 0, 4, st));
        qsim_ctmc_kernel<<<(cfg->R + threads - 1u) / threads, threads, smem, st>>>(p);
        CUDA_TRY(cudaGetLastError());
        ++n;
        CUDA_TRY(cudaMemcpyAsync(&flag, p.not_done, 4, cudaMemcpyDeviceToHost, st));
        CUDA_TRY(cudaStreamSynchronize(st));
    }
    if (launches) *launches = n;
    if (flag != 0) return fail(QSIM_EOVERFLOW, "replications still unfinished after 100000 launches: the end time was not reached");
    return QSIM_OK;
}

int qsim_ctmc_stats(const qsim_ctmc_config *cfg, const void *dev_workspace, size_t bytes, void *cuda_stream, qsim_ctmc_rep_stats *per_rep)
{
    if (!cfg || !per_rep) return fail(QSIM_EINVAL, "null argument");
    if (cfg->size != sizeof(qsim_ctmc_config) || cfg->R < 1 || cfg->qcap < 1 || cfg->I < 1 || cfg->I > QSIM_MAXI) return fail(QSIM_EINVAL, "bad qsim_ctmc_config");
    const CtmcSections sec = ctmc_sections(*cfg);
    if (!dev_workspace || bytes < sec.total) return fail(QSIM_EWORKSPACE, "workspace missing or too small");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    std::vector<CtmcRep> reps(cfg->R);
    CUDA_TRY(cudaMemcpyAsync(reps.data(), static_cast<const char *>(dev_workspace) + sec.reps, reps.size() * sizeof(CtmcRep), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    for (uint32_t r = 0; r < cfg->R; ++r) {
        const CtmcRep &S = reps[r];
        if (S.err) return fail(QSIM_EOVERFLOW, "replication " + std::to_string(r) + " stopped on an internal error");
        qsim_ctmc_rep_stats &o = per_rep[r];
        std::memset(&o, 0, sizeof o);
        const double T = S.T_end;
        for (uint32_t i = 0; i < cfg->I; ++i) {
            for (int k = 0; k < CC_N; ++k) o.cnt[i][k] = S.cnt[i][k];
            const uint32_t state[5] = { S.Qp[i], S.X[i], S.Qd[0][i] + S.Qd[1][i], S.Ym[i], S.Ys[i] };
            for (int a = 0; a < CA_N; ++a) {
                o.state[i][a] = state[a];
                o.area[i][a] = S.area[a][i] + (double)state[a] * (T - S.area_t[a][i]);     // integral up to the end time
            }
        }
        o.events = S.events;
        o.T_elapsed = T;
    }
    return QSIM_OK;
}

int qsim_ctmc_revenue(const qsim_ctmc_config *cfg, const qsim_ctmc_rep_stats *per_rep, const double *P, const double *D,
                      const double *prices, int separate, double *rate)
{
    if (!cfg || !per_rep || !P || !D || !prices || !rate) return fail(QSIM_EINVAL, "null argument");
    if (cfg->size != sizeof(qsim_ctmc_config) || cfg->I < 1 || cfg->I > QSIM_MAXI || cfg->N < 1) return fail(QSIM_EINVAL, "bad qsim_ctmc_config");
    for (uint32_t r = 0; r < cfg->R; ++r) {
        const qsim_ctmc_rep_stats &s = per_rep[r];
        if (!(s.T_elapsed > 0.0)) return fail(QSIM_ESTATE, "no simulated time has elapsed");
        double rev = 0.0;
        for (uint32_t i = 0; i < cfg->I; ++i) {
            const double done = (double)(s.cnt[i][CC_DONE_MIXED] + s.cnt[i][CC_DONE_SOLO]);
            const double paid_in = separate ? (double)s.cnt[i][CC_PREFILL_DONE] : done;       // separate charging credits the prompt at prefill completion
            rev += prices[0] * P[i] * paid_in + prices[1] * D[i] * done;
        }
        rate[r] = rev / ((double)cfg->N * s.T_elapsed);
    }
    return QSIM_OK;
}

}  // extern "C"
