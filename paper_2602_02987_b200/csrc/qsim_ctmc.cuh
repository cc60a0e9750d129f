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
#pragma once

namespace qsimdev {

enum { CK_ARR = 0, CK_ABP = 1, CK_ABD0 = 2, CK_ABD1 = 3, CK_SP = 4, CK_SDM = 5, CK_SDS = 6, CK_N = 7 };
enum { CC_ARRIVALS = 0, CC_ADMITTED, CC_PREFILL_DONE, CC_PLACED_MIXED, CC_PLACED_SOLO, CC_DONE_MIXED, CC_DONE_SOLO,
       CC_ABANDONED_P, CC_ABANDONED_D, CC_OVERFLOW_D, CC_N };
enum { CA_QP = 0, CA_X, CA_QD, CA_YM, CA_YS, CA_N };

struct CtmcClk { double acc, lvl, t_last, t_fire; unsigned long long m; };

// state of one replication (global memory between launches, thread-local while a launch runs)
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

struct CtmcSim {
    const CtmcParams &p;
    CtmcRep &S;
    uint8_t *ring0, *ring1;
    const uint32_t rep;
    uint32_t totX, totYm, totYs;

    __device__ CtmcSim(const CtmcParams &p_, CtmcRep &S_, uint32_t rep_)
        : p(p_), S(S_), ring0(p_.rings + (size_t)rep_ * 2 * p_.qcap), ring1(ring0 + p_.qcap), rep(rep_), totX(0), totYm(0), totYs(0) {}

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
    __device__ __forceinline__ double coef(uint32_t k, uint32_t i) const
    {
        const CtmcClassPar &c = p.cls[i];
        return k <= CK_ABD1 ? (k == CK_ARR ? 0.0 : c.theta) : (k == CK_SP ? c.mu_p : (k == CK_SDM ? c.mu_m : c.mu_s));
    }
    __device__ __forceinline__ void touch(uint32_t a, uint32_t i, uint32_t count, double t)
    {
        S.area[a][i] = __dadd_rn(S.area[a][i], __dmul_rn((double)count, __dsub_rn(t, S.area_t[a][i])));
        S.area_t[a][i] = t;
    }
    // the count that process k of class i runs on changes from n_old to n_new at time t
    __device__ void clk_change(uint32_t k, uint32_t i, uint32_t n_old, uint32_t n_new, double t)
    {
        const double c = coef(k, i);
        if (!(c > 0.0)) return;
        CtmcClk &q = S.clk[k][i];
        q.acc = __dadd_rn(q.acc, __dmul_rn(__dmul_rn(c, (double)n_old), __dsub_rn(t, q.t_last)));
        q.t_last = t;
        if (n_new > 0) {
            double rem = __dsub_rn(q.lvl, q.acc);
            if (rem < 0.0) rem = 0.0;
            q.t_fire = __dadd_rn(t, __ddiv_rn(rem, __dmul_rn(c, (double)n_new)));
        } else {
            q.t_fire = dinf();
        }
    }
    // process k of class i has just jumped at t and its count is now n_new: next level from draw m
    __device__ void clk_fired(uint32_t k, uint32_t i, uint32_t n_new, double t, uint32_t &w2)
    {
        CtmcClk &q = S.clk[k][i];
        uint32_t w0, w1, w3;
        rnd(stream_of(k, i), q.m, w0, w1, w2, w3);
        q.lvl = -qlog(u53(w0, w1));
        q.m += 1;
        q.acc = 0.0;
        q.t_last = t;
        q.t_fire = n_new > 0 ? __dadd_rn(t, __ddiv_rn(q.lvl, __dmul_rn(coef(k, i), (double)n_new))) : dinf();
    }
    __device__ void set_Qp(uint32_t i, uint32_t v, double t) { clk_change(CK_ABP, i, S.Qp[i], v, t); touch(CA_QP, i, S.Qp[i], t); S.Qp[i] = v; }
    __device__ void set_X(uint32_t i, uint32_t v, double t) { clk_change(CK_SP, i, S.X[i], v, t); touch(CA_X, i, S.X[i], t); totX += v - S.X[i]; S.X[i] = v; }
    __device__ void set_Qd(uint32_t pool, uint32_t i, uint32_t v, double t)
    {
        clk_change(pool ? CK_ABD1 : CK_ABD0, i, S.Qd[pool][i], v, t);
        touch(CA_QD, i, S.Qd[0][i] + S.Qd[1][i], t);
        S.Qd[pool][i] = v;
    }
    __device__ void set_Ym(uint32_t i, uint32_t v, double t) { clk_change(CK_SDM, i, S.Ym[i], v, t); touch(CA_YM, i, S.Ym[i], t); totYm += v - S.Ym[i]; S.Ym[i] = v; }
    __device__ void set_Ys(uint32_t i, uint32_t v, double t) { clk_change(CK_SDS, i, S.Ys[i], v, t); touch(CA_YS, i, S.Ys[i], t); totYs += v - S.Ys[i]; S.Ys[i] = v; }

    // Section 4.1 occupancy gate (xi_i = (X_i - n x*_i)/x*_i, ties to the largest Q_p,i - n q*_p,i) or the
    // Section 5.1.1 priority gate (smallest static rank); ties to the lowest class index
    __device__ uint32_t gate_class() const
    {
        uint32_t best = NONE32;
        if (p.gate == 1) {
            for (uint32_t i = 0; i < p.I; ++i)
                if (S.Qp[i] > 0 && (best == NONE32 || p.cls[i].prio < p.cls[best].prio)) best = i;
            return best;
        }
        double bxi = 0.0, bdq = 0.0;
        for (uint32_t i = 0; i < p.I; ++i) {
            if (S.Qp[i] == 0 || !(p.cls[i].xstar > 0.0)) continue;
            const double xi = __ddiv_rn(__dsub_rn((double)S.X[i], p.cls[i].nx), p.cls[i].xstar);
            const double dq = __dsub_rn((double)S.Qp[i], p.cls[i].nq);
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
            while (S.n[pool] > 0) {
                bool to_solo;
                if (p.router == 1) {
                    to_solo = pool == 0;
                    if (to_solo ? totYs >= cap_s : totYm >= cap_m) break;
                } else {
                    if (totYs < cap_s) to_solo = true;
                    else if (totYm < cap_m) to_solo = false;
                    else break;
                }
                const uint32_t i = ring[S.head[pool]];
                S.head[pool] = S.head[pool] + 1 == p.qcap ? 0 : S.head[pool] + 1;
                S.n[pool] -= 1;
                set_Qd(pool, i, S.Qd[pool][i] - 1, t);
                if (to_solo) { set_Ys(i, S.Ys[i] + 1, t); S.cnt[i][CC_PLACED_SOLO]++; }
                else         { set_Ym(i, S.Ym[i] + 1, t); S.cnt[i][CC_PLACED_MIXED]++; }
            }
        }
        while (totX < p.M) {
            const uint32_t i = gate_class();
            if (i == NONE32) break;
            set_Qp(i, S.Qp[i] - 1, t);
            set_X(i, S.X[i] + 1, t);
            S.cnt[i][CC_ADMITTED]++;
        }
    }

    __device__ void init()
    {
        for (uint32_t i = 0; i < p.I; ++i) {
            for (uint32_t k = 0; k < CK_N; ++k) {
                CtmcClk &q = S.clk[k][i];
                uint32_t w0, w1, w2, w3;
                rnd(stream_of(k, i), 0, w0, w1, w2, w3);
                q.acc = 0.0; q.t_last = 0.0; q.t_fire = dinf(); q.lvl = -qlog(u53(w0, w1)); q.m = 1;
            }
            const double Lam = __dmul_rn((double)p.N, p.cls[i].lambda);
            if (Lam > 0.0) S.clk[CK_ARR][i].t_fire = __dadd_rn(0.0, __ddiv_rn(S.clk[CK_ARR][i].lvl, Lam));
        }
    }

    // events with t <= T_end, at most `budget` of them; returns true when none is left up to T_end
    __device__ bool run(double T_end, unsigned long long budget)
    {
        for (uint32_t i = 0; i < p.I; ++i) { totX += S.X[i]; totYm += S.Ym[i]; totYs += S.Ys[i]; }
        S.T_end = T_end;
        for (;;) {
            // earliest process; ties by process kind, then class (strict '<' in that scan order)
            double te = dinf();
            uint32_t bk = 0, bi = 0;
            for (uint32_t k = 0; k < CK_N; ++k)
                for (uint32_t i = 0; i < p.I; ++i) {
                    const double tf = S.clk[k][i].t_fire;
                    if (tf < te) { te = tf; bk = k; bi = i; }
                }
            if (!(te <= T_end)) return true;
            if (budget == 0) return false;
            --budget;
            const double t = te;
            const uint32_t i = bi;
            S.events++;
            uint32_t w2 = 0;
            if (bk == CK_ARR) {
                S.cnt[i][CC_ARRIVALS]++;
                set_Qp(i, S.Qp[i] + 1, t);
                CtmcClk &q = S.clk[CK_ARR][i];
                uint32_t w0, w1, w3;
                rnd(stream_of(CK_ARR, i), q.m, w0, w1, w2, w3);
                q.lvl = -qlog(u53(w0, w1));
                q.m += 1;
                q.t_fire = __dadd_rn(t, __ddiv_rn(q.lvl, __dmul_rn((double)p.N, p.cls[i].lambda)));
            } else if (bk == CK_ABP) {
                touch(CA_QP, i, S.Qp[i], t);
                S.Qp[i] -= 1;
                S.cnt[i][CC_ABANDONED_P]++;
                clk_fired(CK_ABP, i, S.Qp[i], t, w2);
            } else if (bk == CK_ABD0 || bk == CK_ABD1) {
                const uint32_t pool = bk == CK_ABD1 ? 1u : 0u;
                const uint32_t Q = S.Qd[pool][i];
                clk_fired(bk, i, Q - 1, t, w2);
                // a uniformly chosen waiting class-i request leaves the pool's buffer; the rest keep their order
                uint8_t *ring = pool ? ring1 : ring0;
                uint32_t rank = __umulhi(w2, Q), pos = 0;
                const uint32_t n = S.n[pool], head = S.head[pool];
                for (pos = 0; pos < n; ++pos) {
                    uint32_t a = head + pos; if (a >= p.qcap) a -= p.qcap;
                    if (ring[a] != i) continue;
                    if (rank == 0) break;
                    --rank;
                }
                if (pos >= n) { S.err = ERR_INTERNAL; return true; }
                for (uint32_t k = pos; k + 1 < n; ++k) {
                    uint32_t a = head + k, b = head + k + 1;
                    if (a >= p.qcap) a -= p.qcap;
                    if (b >= p.qcap) b -= p.qcap;
                    ring[a] = ring[b];
                }
                S.n[pool] = n - 1;
                touch(CA_QD, i, S.Qd[0][i] + S.Qd[1][i], t);
                S.Qd[pool][i] = Q - 1;
                S.cnt[i][CC_ABANDONED_D]++;
            } else if (bk == CK_SP) {
                touch(CA_X, i, S.X[i], t);
                S.X[i] -= 1; totX -= 1;
                S.cnt[i][CC_PREFILL_DONE]++;
                clk_fired(CK_SP, i, S.X[i], t, w2);
                uint32_t pool = 0;
                if (p.router == 1) {
                    // SLI-aware router: one uniform per finished prefill decides the pool (Section 5.2)
                    uint32_t w0, w1, w3;
                    rnd((STREAM_SLI << 8) | i, S.sli_ord[i]++, w0, w1, w2, w3);
                    pool = u53(w0, w1) <= p.cls[i].ps ? 0u : 1u;
                }
                if (S.n[pool] >= p.qcap) {
                    S.cnt[i][CC_OVERFLOW_D]++;
                } else {
                    uint32_t a = S.head[pool] + S.n[pool]; if (a >= p.qcap) a -= p.qcap;
                    (pool ? ring1 : ring0)[a] = (uint8_t)i;
                    S.n[pool] += 1;
                    set_Qd(pool, i, S.Qd[pool][i] + 1, t);
                }
            } else if (bk == CK_SDM) {
                touch(CA_YM, i, S.Ym[i], t);
                S.Ym[i] -= 1; totYm -= 1;
                S.cnt[i][CC_DONE_MIXED]++;
                clk_fired(CK_SDM, i, S.Ym[i], t, w2);
            } else {
                touch(CA_YS, i, S.Ys[i], t);
                S.Ys[i] -= 1; totYs -= 1;
                S.cnt[i][CC_DONE_SOLO]++;
                clk_fired(CK_SDS, i, S.Ys[i], t, w2);
            }
            dispatch(t);
        }
    }
};

// One thread per replication, working on its record in global memory (a few KB that stay in the L1/L2 caches
// while the thread runs).  init != 0: start from the empty system at t = 0 (no events are processed).
__global__ void __launch_bounds__(64) qsim_ctmc_kernel(CtmcParams p)
{
    const uint32_t rep = blockIdx.x * blockDim.x + threadIdx.x;
    if (rep >= p.R) return;
    CtmcRep &S = p.reps[rep];
    if (p.init) {
        uint32_t *w = reinterpret_cast<uint32_t *>(&S);
        for (uint32_t o = 0; o < sizeof(CtmcRep) / 4; ++o) w[o] = 0;
        CtmcSim sim(p, S, rep);
        sim.init();
        S.done = 1;
        return;
    }
    if (S.err || (S.done && S.T_end == p.T_end)) return;
    CtmcSim sim(p, S, rep);
    const bool finished = sim.run(p.T_end, p.event_budget);
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
    qsim_ctmc_kernel<<<(cfg->R + 63u) / 64u, 64, 0, st>>>(p);
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
    // a replication that used up its per-launch event budget is continued by further launches
    for (int guard = 0; guard < 100000; ++guard) {
        uint32_t flag = 0;
        CUDA_TRY(cudaMemsetAsync(p.not_done, 0, 4, st));
        qsim_ctmc_kernel<<<(cfg->R + 63u) / 64u, 64, 0, st>>>(p);
        CUDA_TRY(cudaGetLastError());
        ++n;
        CUDA_TRY(cudaMemcpyAsync(&flag, p.not_done, 4, cudaMemcpyDeviceToHost, st));
        CUDA_TRY(cudaStreamSynchronize(st));
        if (flag == 0) break;
    }
    if (launches) *launches = n;
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

}  // extern "C"
