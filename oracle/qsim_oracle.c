/*
 * CPU oracle of the many-replication gate-and-route simulation.  TEST INFRASTRUCTURE ONLY:
 * see qsim_oracle.h for scope, citations and pins.  Compile with -ffp-contract=off so that
 * every floating-point operation below is one IEEE-754 double operation rounded to nearest.
 */
#include "qsim_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------
 * Counter-based random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
 * Ten rounds; each round multiplies counter words 0 and 2 by two fixed 32-bit constants, mixes the
 * high halves with the other two words and the round key, and the key advances by Weyl constants.
 * ------------------------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Uniform on (0,1] with 53 random bits: (h + 1) / 2^53, h = top 53 bits of (w0:w1). */
double orc_u53(uint32_t w0, uint32_t w1)
{
    uint64_t h = ((uint64_t)w0 << 21) | (uint64_t)(w1 >> 11);
    return (double)(h + 1) * 0x1.0p-53;
}

/*
 * Natural logarithm as a fixed sequence of IEEE operations (no libm): x = m 2^e with
 * m in [sqrt(1/2), sqrt(2)), s = (m-1)/(m+1), log m = 2 s (1 + s^2/3 + s^4/5 + ... + s^24/25).
 * Not correctly rounded (error about 1e-16); what matters is that the operation order is fixed.
 */
double orc_qlog(double x)
{
    uint64_t bits;
    memcpy(&bits, &x, sizeof bits);
    int e = (int)((bits >> 52) & 0x7FF) - 1023;
    bits = (bits & 0x000FFFFFFFFFFFFFull) | 0x3FF0000000000000ull;
    double m;
    memcpy(&m, &bits, sizeof m);                /* m in [1,2) */
    if (m > 0x1.6a09e667f3bcdp+0) {             /* sqrt(2) */
        m = m * 0.5;
        e += 1;
    }
    double s = (m - 1.0) / (m + 1.0);
    double z = s * s;
    double p = 1.0 / 25.0;
    for (int k = 11; k >= 0; --k)
        p = p * z + 1.0 / (double)(2 * k + 1);
    double logm = (2.0 * s) * p;
    return (double)e * 0x1.62e42fefa39efp-1 + logm;   /* ln 2 */
}

/*
 * Iteration time (Eq. (1)-(3), six-coefficient family):
 *   prefill chunk present:  alpha_m + beta p + delta_m d        (tau_mix(C) = alpha + beta C when delta_m = 0)
 *   decode only:            alpha_s + delta_s d                 (tau_solo = c when delta_s = 0)
 *   plus kappa K when kappa != 0 (K = KV tokens resident on the GPU; Section 6.1 solo fit).
 */
double orc_tau(const double c[6], uint32_t p, uint32_t d, uint64_t K)
{
    double t;
    if (p > 0) {
        t = c[0] + c[1] * (double)p;
        t = t + c[2] * (double)d;
    } else {
        t = c[3] + c[4] * (double)d;
    }
    if (c[5] != 0.0)
        t = t + c[5] * (double)K;
    return t;
}

/* len = 1 + #{ j in [0, LMAX-1) : thr[j] <= w } for a non-decreasing threshold table. */
uint32_t orc_table_length(const uint32_t *thr, uint32_t w)
{
    uint32_t n = 0;
    for (uint32_t j = 0; j < ORC_LMAX - 1; ++j)
        if (thr[j] <= w)
            ++n;
    return 1 + n;
}

/* Log-linear histogram: 32 sub-bins per octave from 2^-20 s up; bin = top bits of the IEEE pattern. */
uint32_t orc_hist_bin(double x)
{
    uint64_t bits;
    memcpy(&bits, &x, sizeof bits);
    int64_t b = (int64_t)(bits >> 47) - ((int64_t)(1023 - 20) << 5);
    if (b < 0) b = 0;
    if (b > ORC_NBIN - 1) b = ORC_NBIN - 1;
    return (uint32_t)b;
}

/* ------------------------------------------------------------------------------------------ */

enum { STREAM_ARRIVAL = 0, STREAM_ABANDON_P = 1, STREAM_ABANDON_D0 = 2, STREAM_ABANDON_D1 = 3,
       STREAM_PLACEMENT = 4, STREAM_SLI = 5, STREAM_SELECT0 = 6, STREAM_SELECT1 = 7 };

typedef struct { double t_arr; uint32_t P, D; uint64_t ord; } job_t;
typedef struct { double t_pf; uint32_t P, D, cls; uint64_t ord; } djob_t;
typedef struct { int used, mixed; uint32_t finish_it; djob_t j; } slot_t;

typedef struct {
    int running;
    double t_next, tau_cur;
    uint32_t it, n_dec, n_act;
    int pf_present;
    uint32_t pf_cls, pf_rem, pf_cur;
    job_t pf_job;
    uint64_t K, K_pend;
    slot_t *slots;
} server_t;

typedef struct { double acc, lvl, t_last, t_ab; uint64_t m; } abclock_t;
typedef struct { double area, t_last; } area_t;

typedef struct {
    double T_end, T_reset;
    uint64_t H_total;           /* iterations of horizon requested so far: T_end = H_total * tau_ref */
    uint32_t blk;
    /* arrivals */
    double ta[ORC_MAXI];
    uint64_t adraw[ORC_MAXI], aord[ORC_MAXI];
    uint32_t ablk[ORC_MAXI], nextP[ORC_MAXI], nextD[ORC_MAXI];
    uint32_t inj_pos[ORC_MAXI];
    /* prefill queues (FCFS per class) and decode buffers (pool 0: single / solo, pool 1: mixed) */
    job_t *pq[ORC_MAXI];
    uint32_t pq_n[ORC_MAXI];
    djob_t *dq[2];
    uint32_t dq_n[2];
    uint32_t Qd_pool[2][ORC_MAXI];
    abclock_t abp[ORC_MAXI], abd[2][ORC_MAXI];
    server_t *srv;
    uint64_t place_ord, sli_ord[ORC_MAXI], sel_ord[2];
    /* state counts and their time integrals */
    uint32_t X[ORC_MAXI], Ym[ORC_MAXI], Ys[ORC_MAXI];
    area_t aQp[ORC_MAXI], aX[ORC_MAXI], aQd[ORC_MAXI], aYm[ORC_MAXI], aYs[ORC_MAXI];
    orc_rep_stats st;
    uint64_t *h_ttft, *h_tpot;   /* [I][NBIN] or NULL */
} rep_t;

struct orc_sim {
    orc_config cfg;
    orc_class cls[ORC_MAXI];
    double *rates;
    uint32_t *lengths;
    double prices[2], coeffs[6];
    orc_targets *tg;
    double *inj_t;
    uint32_t *inj_job;
    rep_t *reps;
    orc_trace_rec *trace;
    uint64_t trace_cap, trace_n;
};

static void trace(orc_sim *s, uint32_t r, int type, double t, int cls, int server, uint64_t job, double aux)
{
    if (!s->trace) return;
    if (s->trace_n < s->trace_cap) {
        orc_trace_rec *e = &s->trace[s->trace_n];
        e->t = t; e->aux = aux; e->job = job; e->type = type; e->cls = cls; e->server = server; e->rep = (int32_t)r;
    }
    s->trace_n++;
}

static void draw(const orc_sim *s, uint32_t r, uint32_t stream, uint64_t index, uint32_t w[4])
{
    uint64_t rep = s->cfg.rep_offset + r;
    uint32_t ctr[4] = { (uint32_t)index, (uint32_t)(index >> 32), stream, (uint32_t)rep };
    uint32_t key[2] = { (uint32_t)s->cfg.seed, (uint32_t)(s->cfg.seed >> 32) };
    orc_philox4x32_10(ctr, key, w);
}

static double block_start(const orc_sim *s, uint32_t b) { return (double)b * s->cfg.block_len; }

static void area_touch(area_t *a, uint32_t count, double t)
{
    a->area = a->area + (double)count * (t - a->t_last);
    a->t_last = t;
}

/* Abandonment through the time change of Eq. (8)-(9): B(t) = N(int theta Q ds) with N a unit-rate
 * Poisson process.  acc is the integral since the last jump, lvl the exponential gap to the next. */
static void ab_change(abclock_t *c, double theta, uint32_t Q_old, uint32_t Q_new, double t)
{
    if (!(theta > 0.0)) return;
    c->acc = c->acc + (theta * (double)Q_old) * (t - c->t_last);
    c->t_last = t;
    if (Q_new > 0) {
        double rem = c->lvl - c->acc;
        if (rem < 0.0) rem = 0.0;
        c->t_ab = t + rem / (theta * (double)Q_new);
    } else {
        c->t_ab = INFINITY;
    }
}

/* Schedule the next class-i arrival after time t0 (Poisson, rate N*lambda_i of the block that holds
 * t0).  A candidate at or past the block's end is discarded and the draw is repeated from the block
 * boundary under the next block's rate (memorylessness). */
static void schedule_arrival(orc_sim *s, uint32_t r, uint32_t i, double t0)
{
    rep_t *R = &s->reps[r];
    const orc_config *c = &s->cfg;
    if (c->n_inject > 0) {
        uint32_t k = R->inj_pos[i];
        while (k < c->n_inject && s->inj_job[3 * k] != i) ++k;
        if (k < c->n_inject) {
            R->ta[i] = s->inj_t[k];
            R->nextP[i] = s->inj_job[3 * k + 1];
            R->nextD[i] = s->inj_job[3 * k + 2];
            R->inj_pos[i] = k + 1;
        } else {
            R->ta[i] = INFINITY;
            R->inj_pos[i] = k;
        }
        return;
    }
    for (;;) {
        uint32_t b = R->ablk[i];
        double Lam = (double)c->N * s->rates[(size_t)b * c->I + i];
        int has_next = b + 1 < c->nblk;
        if (!(Lam > 0.0)) {
            if (!has_next) { R->ta[i] = INFINITY; return; }
            R->ablk[i] = b + 1;
            t0 = block_start(s, b + 1);
            continue;
        }
        uint32_t w[4];
        draw(s, r, (STREAM_ARRIVAL << 8) | i, R->adraw[i]++, w);
        double E = -orc_qlog(orc_u53(w[0], w[1]));
        double cand = t0 + E / Lam;
        if (has_next && cand >= block_start(s, b + 1)) {
            R->ablk[i] = b + 1;
            t0 = block_start(s, b + 1);
            continue;
        }
        R->ta[i] = cand;
        if (c->length_mode == 1) {
            R->nextP[i] = orc_table_length(s->lengths + ((size_t)i * 2 + 0) * ORC_LMAX, w[2]);
            R->nextD[i] = orc_table_length(s->lengths + ((size_t)i * 2 + 1) * ORC_LMAX, w[3]);
        } else {
            R->nextP[i] = s->cls[i].P;
            R->nextD[i] = s->cls[i].D;
        }
        return;
    }
}

static uint32_t decode_cap(const orc_sim *s, const rep_t *R, uint32_t g)
{
    /* A mixed GPU keeps one slot for prefill (Section 4.1, Static Planning; Eq. (13)-(14)). */
    uint32_t M = s->tg[R->blk].M;
    return (g < M || R->srv[g].pf_present) ? s->cfg.B - 1 : s->cfg.B;
}

/* eligibility predicates of the three placement decisions */
enum { WANT_SOLO_DECODE, WANT_MIX_DECODE, WANT_PREFILL };
static int eligible(const orc_sim *s, const rep_t *R, uint32_t g, int want)
{
    uint32_t M = s->tg[R->blk].M;
    const server_t *v = &R->srv[g];
    switch (want) {
    case WANT_SOLO_DECODE: return g >= M && v->n_dec < decode_cap(s, R, g);
    case WANT_MIX_DECODE:  return g < M && v->n_dec < decode_cap(s, R, g);
    default:               return g < M && !v->pf_present && v->n_dec <= s->cfg.B - 1;
    }
}

/* Pick one GPU of the eligible set: uniformly at random (paper) or least loaded, lowest index. */
static int choose_server(orc_sim *s, uint32_t r, int want)
{
    rep_t *R = &s->reps[r];
    uint32_t N = s->cfg.N, cnt = 0;
    for (uint32_t g = 0; g < N; ++g)
        if (eligible(s, R, g, want)) ++cnt;
    if (cnt == 0) return -1;
    if (s->cfg.placement == 0) {
        uint32_t idx = 0;
        if (cnt > 1) {
            uint32_t w[4];
            draw(s, r, STREAM_PLACEMENT << 8, R->place_ord++, w);
            idx = (uint32_t)(((uint64_t)w[0] * cnt) >> 32);
        }
        for (uint32_t g = 0; g < N; ++g)
            if (eligible(s, R, g, want)) {
                if (idx == 0) return (int)g;
                --idx;
            }
        return -1;
    }
    int best = -1;
    for (uint32_t g = 0; g < N; ++g)
        if (eligible(s, R, g, want) && (best < 0 || R->srv[g].n_dec < R->srv[best].n_dec))
            best = (int)g;
    return best;
}

/* entry `pos` of the pool's buffer (0 = head) starts decoding on GPU g */
static void place_decode(orc_sim *s, uint32_t r, uint32_t pool, uint32_t g, uint32_t pos, double t)
{
    rep_t *R = &s->reps[r];
    server_t *v = &R->srv[g];
    djob_t j = R->dq[pool][pos];
    memmove(R->dq[pool] + pos, R->dq[pool] + pos + 1, (size_t)(R->dq_n[pool] - 1 - pos) * sizeof(djob_t));
    uint32_t i = j.cls;
    ab_change(&R->abd[pool][i], s->cls[i].theta, R->Qd_pool[pool][i], R->Qd_pool[pool][i] - 1, t);
    area_touch(&R->aQd[i], R->Qd_pool[0][i] + R->Qd_pool[1][i], t);
    R->dq_n[pool]--;
    R->Qd_pool[pool][i]--;
    uint32_t sl = 0;
    while (v->slots[sl].used) ++sl;
    int mixed = g < s->tg[R->blk].M;
    v->slots[sl].used = 1;
    v->slots[sl].mixed = mixed;
    v->slots[sl].j = j;
    /* joins the iteration that starts next: the running one finishes as it+1 first */
    v->slots[sl].finish_it = v->it + (v->running ? 1u : 0u) + j.D;
    v->n_dec++;
    v->K_pend += j.P;
    if (mixed) { area_touch(&R->aYm[i], R->Ym[i], t); R->Ym[i]++; R->st.cls[i].placed_mixed++; }
    else       { area_touch(&R->aYs[i], R->Ys[i], t); R->Ys[i]++; R->st.cls[i].placed_solo++; }
    trace(s, r, ORC_EV_PLACE, t, (int)i, (int)g, j.ord, 0.0);
}

/* Prefill gate: which waiting class goes next (Section 4.1 occupancy gate / Section 5.1.1 priority). */
static int gate_class(const orc_sim *s, const rep_t *R)
{
    const orc_targets *tg = &s->tg[R->blk];
    int best = -1;
    if (s->cfg.gate == 2) {
        /* ablation "FCFS-and-Route" (EC, additional ablation studies): no class rule, the oldest waiting request goes first */
        for (uint32_t i = 0; i < s->cfg.I; ++i)
            if (R->pq_n[i] > 0 && (best < 0 || R->pq[i][0].t_arr < R->pq[best][0].t_arr))
                best = (int)i;
        return best;
    }
    if (s->cfg.gate == 1) {
        for (uint32_t i = 0; i < s->cfg.I; ++i)
            if (R->pq_n[i] > 0 && (best < 0 || s->cls[i].prio_rank < s->cls[best].prio_rank))
                best = (int)i;
        return best;
    }
    double best_xi = 0.0, best_dq = 0.0;
    for (uint32_t i = 0; i < s->cfg.I; ++i) {
        if (R->pq_n[i] == 0 || !(tg->xstar[i] > 0.0)) continue;
        double xi = ((double)R->X[i] - tg->n_xstar[i]) / tg->xstar[i];      /* xi_i = (X_i - n x*_i) / x*_i */
        double dq = (double)R->pq_n[i] - tg->n_qpstar[i];                     /* Q_p,i - n q*_p,i */
        if (best < 0 || xi < best_xi || (xi == best_xi && dq > best_dq)) {
            best = (int)i; best_xi = xi; best_dq = dq;
        }
    }
    return best;
}

static void start_iteration(orc_sim *s, rep_t *R, uint32_t g, double t)
{
    server_t *v = &R->srv[g];
    v->K += v->K_pend;
    v->K_pend = 0;
    v->n_act = v->n_dec;
    v->pf_cur = v->pf_present ? (v->pf_rem < s->cfg.C ? v->pf_rem : s->cfg.C) : 0;
    v->tau_cur = orc_tau(s->coeffs, v->pf_cur, v->n_act, v->K);
    v->t_next = t + v->tau_cur;
    v->running = 1;
}

/* General SLI-aware router: when a slot of the pool frees up, the class is drawn with probabilities
 * proportional to varpi restricted to the classes that wait in the pool's buffer; its oldest request goes.
 * One waiting class needs no draw; if every waiting class has weight 0 the oldest request of the buffer goes. */
static uint32_t select_in_pool(orc_sim *s, uint32_t r, uint32_t pool)
{
    rep_t *R = &s->reps[r];
    const orc_targets *tg = &s->tg[R->blk];
    const double *w = pool == 0 ? tg->w_solo : tg->w_mix;
    uint32_t I = s->cfg.I, nonempty = 0, only = 0;
    double Wsum = 0.0;
    for (uint32_t i = 0; i < I; ++i)
        if (R->Qd_pool[pool][i] > 0) { ++nonempty; only = i; Wsum = Wsum + w[i]; }
    uint32_t cls = only;
    if (nonempty > 1) {
        if (!(Wsum > 0.0)) return 0;
        uint32_t wd[4];
        draw(s, r, (pool == 0 ? STREAM_SELECT0 : STREAM_SELECT1) << 8, R->sel_ord[pool]++, wd);
        double x = orc_u53(wd[0], wd[1]) * Wsum, cum = 0.0;
        int chosen = -1, last = -1;
        for (uint32_t i = 0; i < I && chosen < 0; ++i) {
            if (R->Qd_pool[pool][i] == 0) continue;
            cum = cum + w[i];
            if (w[i] > 0.0) last = (int)i;
            if (w[i] > 0.0 && cum >= x) chosen = (int)i;
        }
        cls = (uint32_t)(chosen >= 0 ? chosen : last);
    }
    uint32_t pos = 0;
    while (R->dq[pool][pos].cls != cls) ++pos;
    return pos;
}

static void dispatch(orc_sim *s, uint32_t r, double t)
{
    rep_t *R = &s->reps[r];
    const orc_config *c = &s->cfg;
    /* decode routing: buffered jobs first (FCFS), solo GPUs before mixed ones */
    if (c->router == 0 || c->router == 3) {      /* router 3 never leaves a request in the buffer */
        while (R->dq_n[0] > 0) {
            int g = choose_server(s, r, WANT_SOLO_DECODE);
            if (g < 0) g = choose_server(s, r, WANT_MIX_DECODE);
            if (g < 0) break;
            place_decode(s, r, 0, (uint32_t)g, 0, t);
        }
    } else {
        for (uint32_t pool = 0; pool < 2; ++pool)
            while (R->dq_n[pool] > 0) {
                int g = choose_server(s, r, pool == 0 ? WANT_SOLO_DECODE : WANT_MIX_DECODE);
                if (g < 0) break;
                place_decode(s, r, pool, (uint32_t)g, c->router == 2 ? select_in_pool(s, r, pool) : 0u, t);
            }
    }
    /* prefill gate on the mixed GPUs whose prefill slot is idle */
    for (;;) {
        int i = gate_class(s, R);
        if (i < 0) break;
        int g = choose_server(s, r, WANT_PREFILL);
        if (g < 0) break;
        job_t j = R->pq[i][0];
        memmove(R->pq[i], R->pq[i] + 1, (size_t)(R->pq_n[i] - 1) * sizeof(job_t));
        ab_change(&R->abp[i], s->cls[i].theta, R->pq_n[i], R->pq_n[i] - 1, t);
        area_touch(&R->aQp[i], R->pq_n[i], t);
        R->pq_n[i]--;
        area_touch(&R->aX[i], R->X[i], t);
        R->X[i]++;
        R->st.cls[i].admitted++;
        server_t *v = &R->srv[g];
        v->pf_present = 1;
        v->pf_cls = (uint32_t)i;
        v->pf_rem = j.P;
        v->pf_job = j;
        trace(s, r, ORC_EV_ADMIT, t, i, g, j.ord, 0.0);
    }
    /* every GPU that has work and is between iterations starts its next iteration now */
    for (uint32_t g = 0; g < c->N; ++g) {
        server_t *v = &R->srv[g];
        if (!v->running && (v->n_dec > 0 || v->pf_present))
            start_iteration(s, R, g, t);
    }
}

static void on_arrival(orc_sim *s, uint32_t r, uint32_t i, double t)
{
    rep_t *R = &s->reps[r];
    uint64_t ord = R->aord[i]++;
    R->st.cls[i].arrivals++;
    trace(s, r, ORC_EV_ARRIVAL, t, (int)i, -1, ord, 0.0);
    if (R->pq_n[i] >= s->cfg.qcap) {
        R->st.cls[i].overflow++;
        trace(s, r, ORC_EV_OVERFLOW, t, (int)i, -1, ord, 0.0);
    } else {
        ab_change(&R->abp[i], s->cls[i].theta, R->pq_n[i], R->pq_n[i] + 1, t);
        area_touch(&R->aQp[i], R->pq_n[i], t);
        job_t *j = &R->pq[i][R->pq_n[i]++];
        j->t_arr = t; j->P = R->nextP[i]; j->D = R->nextD[i]; j->ord = ord;
    }
    schedule_arrival(s, r, i, t);
}

/* One waiting class-i job, uniformly chosen in FCFS rank, leaves the prefill queue (Eq. (8)). */
static void on_abandon_p(orc_sim *s, uint32_t r, uint32_t i, double t)
{
    rep_t *R = &s->reps[r];
    abclock_t *c = &R->abp[i];
    uint32_t Q = R->pq_n[i], w[4];
    draw(s, r, (STREAM_ABANDON_P << 8) | i, c->m++, w);
    uint32_t rank = (uint32_t)(((uint64_t)w[2] * Q) >> 32);
    trace(s, r, ORC_EV_ABANDON_P, t, (int)i, -1, R->pq[i][rank].ord, 0.0);
    memmove(R->pq[i] + rank, R->pq[i] + rank + 1, (size_t)(Q - 1 - rank) * sizeof(job_t));
    area_touch(&R->aQp[i], Q, t);
    R->pq_n[i] = Q - 1;
    R->st.cls[i].abandoned_p++;
    c->acc = 0.0;
    c->lvl = -orc_qlog(orc_u53(w[0], w[1]));
    c->t_last = t;
    c->t_ab = (Q - 1 > 0) ? t + c->lvl / (s->cls[i].theta * (double)(Q - 1)) : INFINITY;
}

/* Same for the decode buffer of one pool (Eq. (9)). */
static void on_abandon_d(orc_sim *s, uint32_t r, uint32_t pool, uint32_t i, double t)
{
    rep_t *R = &s->reps[r];
    abclock_t *c = &R->abd[pool][i];
    uint32_t Q = R->Qd_pool[pool][i], w[4];
    draw(s, r, ((pool == 0 ? STREAM_ABANDON_D0 : STREAM_ABANDON_D1) << 8) | i, c->m++, w);
    uint32_t rank = (uint32_t)(((uint64_t)w[2] * Q) >> 32);
    uint32_t pos = 0;
    for (;; ++pos)
        if (R->dq[pool][pos].cls == i) {
            if (rank == 0) break;
            --rank;
        }
    trace(s, r, ORC_EV_ABANDON_D, t, (int)i, -1, R->dq[pool][pos].ord, 0.0);
    memmove(R->dq[pool] + pos, R->dq[pool] + pos + 1, (size_t)(R->dq_n[pool] - 1 - pos) * sizeof(djob_t));
    area_touch(&R->aQd[i], R->Qd_pool[0][i] + R->Qd_pool[1][i], t);
    R->dq_n[pool]--;
    R->Qd_pool[pool][i] = Q - 1;
    R->st.cls[i].abandoned_d++;
    c->acc = 0.0;
    c->lvl = -orc_qlog(orc_u53(w[0], w[1]));
    c->t_last = t;
    c->t_ab = (Q - 1 > 0) ? t + c->lvl / (s->cls[i].theta * (double)(Q - 1)) : INFINITY;
}

/* End of an iteration on GPU g: every active decode emitted one token, the prefill advanced one chunk. */
static void on_server(orc_sim *s, uint32_t r, uint32_t g, double t)
{
    rep_t *R = &s->reps[r];
    const orc_config *c = &s->cfg;
    server_t *v = &R->srv[g];
    v->it++;
    v->running = 0;
    v->t_next = INFINITY;
    if (v->pf_cur > 0) { R->st.iters_mixed++; R->st.busy_mixed = R->st.busy_mixed + v->tau_cur; }
    else               { R->st.iters_solo++;  R->st.busy_solo = R->st.busy_solo + v->tau_cur; }
    v->K += v->n_act;
    trace(s, r, ORC_EV_ITER_END, t, -1, (int)g, v->it, v->tau_cur);
    for (uint32_t sl = 0; sl < c->B; ++sl) {
        slot_t *q = &v->slots[sl];
        if (!q->used || q->finish_it != v->it) continue;
        uint32_t i = q->j.cls;
        orc_class_stats *cs = &R->st.cls[i];
        q->used = 0;
        v->n_dec--;
        v->K -= (uint64_t)q->j.P + q->j.D;
        if (q->mixed) { area_touch(&R->aYm[i], R->Ym[i], t); R->Ym[i]--; cs->done_mixed++; }
        else          { area_touch(&R->aYs[i], R->Ys[i], t); R->Ys[i]--; cs->done_solo++; }
        cs->tokens_in_completed += q->j.P;     /* bundled revenue is credited here, Eq. (21)-(22) */
        cs->tokens_out_completed += q->j.D;
        double tpot = (t - q->j.t_pf) / (double)q->j.D;
        cs->sum_tpot = cs->sum_tpot + tpot;
        if (R->h_tpot) R->h_tpot[(size_t)i * ORC_NBIN + orc_hist_bin(tpot)]++;
        trace(s, r, ORC_EV_DECODE_DONE, t, (int)i, (int)g, q->j.ord, 0.0);
    }
    if (v->pf_cur > 0) {
        v->pf_rem -= v->pf_cur;
        if (v->pf_rem == 0) {
            uint32_t i = v->pf_cls;
            orc_class_stats *cs = &R->st.cls[i];
            v->pf_present = 0;
            area_touch(&R->aX[i], R->X[i], t);
            R->X[i]--;
            cs->prefill_done++;
            cs->tokens_in_prefilled += v->pf_job.P;   /* separate charging credits prefill here, Eq. (23) */
            double ttft = t - v->pf_job.t_arr;
            cs->sum_ttft = cs->sum_ttft + ttft;
            if (R->h_ttft) R->h_ttft[(size_t)i * ORC_NBIN + orc_hist_bin(ttft)]++;
            /* hand over to the decode stage: pool drawn once per job under the SLI-aware router */
            uint32_t pool = 0;
            if (c->router == 1 || c->router == 2) {
                uint32_t w[4];
                draw(s, r, (STREAM_SLI << 8) | i, R->sli_ord[i]++, w);
                pool = (orc_u53(w[0], w[1]) <= s->tg[R->blk].p_solo[i]) ? 0u : 1u;
            }
            trace(s, r, ORC_EV_PREFILL_DONE, t, (int)i, (int)g, v->pf_job.ord, (double)pool);   /* aux = pool */
            if (R->dq_n[pool] >= c->qcap) {
                cs->overflow_d++;
                trace(s, r, ORC_EV_OVERFLOW, t, (int)i, (int)g, v->pf_job.ord, 0.0);
            } else {
                ab_change(&R->abd[pool][i], s->cls[i].theta, R->Qd_pool[pool][i], R->Qd_pool[pool][i] + 1, t);
                area_touch(&R->aQd[i], R->Qd_pool[0][i] + R->Qd_pool[1][i], t);
                djob_t *d = &R->dq[pool][R->dq_n[pool]++];
                d->t_pf = t; d->P = v->pf_job.P; d->D = v->pf_job.D; d->cls = i; d->ord = v->pf_job.ord;
                R->Qd_pool[pool][i]++;
                /* ablation "immediate same-slot decoding" (EC, additional ablation studies): no router, the request
                 * goes on decoding on this GPU, in the slot it already holds (it passes through the empty buffer) */
                if (c->router == 3) place_decode(s, r, 0, g, R->dq_n[0] - 1, t);
            }
        }
    }
    v->pf_cur = 0;
}

static void run_rep(orc_sim *s, uint32_t r, double T_end)
{
    rep_t *R = &s->reps[r];
    const orc_config *c = &s->cfg;
    R->T_end = T_end;
    for (;;) {
        /* earliest event; exact ties go to the source listed first: block end, arrivals by class,
         * prefill-queue abandonments by class, decode-buffer abandonments by pool then class, GPUs by index */
        double te = INFINITY;
        int kind = -1;
        uint32_t a = 0, b = 0;
        if (R->blk + 1 < c->nblk) { te = block_start(s, R->blk + 1); kind = 0; }
        for (uint32_t i = 0; i < c->I; ++i) if (R->ta[i] < te) { te = R->ta[i]; kind = 1; a = i; }
        for (uint32_t i = 0; i < c->I; ++i) if (R->abp[i].t_ab < te) { te = R->abp[i].t_ab; kind = 2; a = i; }
        for (uint32_t p = 0; p < 2; ++p)
            for (uint32_t i = 0; i < c->I; ++i)
                if (R->abd[p][i].t_ab < te) { te = R->abd[p][i].t_ab; kind = 3; a = p; b = i; }
        for (uint32_t g = 0; g < c->N; ++g)
            if (R->srv[g].running && R->srv[g].t_next < te) { te = R->srv[g].t_next; kind = 4; a = g; }
        if (kind < 0 || te > T_end) break;
        R->st.events++;
        switch (kind) {
        case 0: R->blk++; trace(s, r, ORC_EV_BLOCK, te, -1, -1, R->blk, 0.0); break;
        case 1: on_arrival(s, r, a, te); break;
        case 2: on_abandon_p(s, r, a, te); break;
        case 3: on_abandon_d(s, r, a, b, te); break;
        default: on_server(s, r, a, te); break;
        }
        dispatch(s, r, te);
    }
}

/* ------------------------------------------------------------------------------------------ */

static double tau_ref(const orc_sim *s) { return orc_tau(s->coeffs, 0, s->cfg.B, 0); }

int orc_create(orc_sim **out, const orc_config *cfg, const orc_class *classes, const double *rates,
               const uint32_t *lengths, const double *prices, const double *coeffs,
               const orc_targets *targets, const double *inject_t, const uint32_t *inject_job)
{
    if (!out || !cfg || !classes || !rates || !prices || !coeffs || !targets) return -1;
    if (cfg->I < 1 || cfg->I > ORC_MAXI || cfg->N < 1 || cfg->R < 1 || cfg->B < 1 || cfg->C < 1 || cfg->nblk < 1 ||
        cfg->qcap < 1)
        return -1;
    if (cfg->length_mode == 1 && !lengths) return -1;
    if (cfg->n_inject > 0 && (!inject_t || !inject_job)) return -1;
    orc_sim *s = (orc_sim *)calloc(1, sizeof *s);
    if (!s) return -2;
    s->cfg = *cfg;
    memcpy(s->cls, classes, cfg->I * sizeof(orc_class));
    size_t nr = (size_t)cfg->nblk * cfg->I;
    s->rates = (double *)malloc(nr * sizeof(double));
    memcpy(s->rates, rates, nr * sizeof(double));
    if (lengths) {
        size_t nl = (size_t)cfg->I * 2 * ORC_LMAX;
        s->lengths = (uint32_t *)malloc(nl * sizeof(uint32_t));
        memcpy(s->lengths, lengths, nl * sizeof(uint32_t));
    }
    memcpy(s->prices, prices, sizeof s->prices);
    memcpy(s->coeffs, coeffs, sizeof s->coeffs);
    s->tg = (orc_targets *)malloc(cfg->nblk * sizeof(orc_targets));
    memcpy(s->tg, targets, cfg->nblk * sizeof(orc_targets));
    if (cfg->n_inject > 0) {
        s->inj_t = (double *)malloc(cfg->n_inject * sizeof(double));
        memcpy(s->inj_t, inject_t, cfg->n_inject * sizeof(double));
        s->inj_job = (uint32_t *)malloc((size_t)cfg->n_inject * 3 * sizeof(uint32_t));
        memcpy(s->inj_job, inject_job, (size_t)cfg->n_inject * 3 * sizeof(uint32_t));
    }
    s->reps = (rep_t *)calloc(cfg->R, sizeof(rep_t));
    for (uint32_t r = 0; r < cfg->R; ++r) {
        rep_t *R = &s->reps[r];
        for (uint32_t i = 0; i < cfg->I; ++i)
            R->pq[i] = (job_t *)calloc(cfg->qcap, sizeof(job_t));
        for (uint32_t p = 0; p < 2; ++p)
            R->dq[p] = (djob_t *)calloc(cfg->qcap, sizeof(djob_t));
        R->srv = (server_t *)calloc(cfg->N, sizeof(server_t));
        for (uint32_t g = 0; g < cfg->N; ++g) {
            R->srv[g].slots = (slot_t *)calloc(cfg->B, sizeof(slot_t));
            R->srv[g].t_next = INFINITY;
        }
        if (cfg->hist) {
            R->h_ttft = (uint64_t *)calloc((size_t)cfg->I * ORC_NBIN, sizeof(uint64_t));
            R->h_tpot = (uint64_t *)calloc((size_t)cfg->I * ORC_NBIN, sizeof(uint64_t));
        }
        for (uint32_t i = 0; i < cfg->I; ++i) {
            abclock_t *clk[3] = { &R->abp[i], &R->abd[0][i], &R->abd[1][i] };
            uint32_t streams[3] = { STREAM_ABANDON_P, STREAM_ABANDON_D0, STREAM_ABANDON_D1 };
            for (int k = 0; k < 3; ++k) {
                uint32_t w[4];
                draw(s, r, (streams[k] << 8) | i, 0, w);
                clk[k]->acc = 0.0;
                clk[k]->lvl = -orc_qlog(orc_u53(w[0], w[1]));
                clk[k]->t_last = 0.0;
                clk[k]->t_ab = INFINITY;
                clk[k]->m = 1;
            }
            schedule_arrival(s, r, i, 0.0);
        }
    }
    *out = s;
    return 0;
}

int orc_set_trace(orc_sim *s, orc_trace_rec *buf, uint64_t cap)
{
    if (!s) return -1;
    s->trace = buf; s->trace_cap = cap; s->trace_n = 0;
    return 0;
}

uint64_t orc_trace_count(const orc_sim *s) { return s ? s->trace_n : 0; }

int orc_run(orc_sim *s, uint64_t horizon_iters, uint32_t rep_lo, uint32_t rep_hi)
{
    if (!s || rep_lo > rep_hi || rep_hi > s->cfg.R) return -1;
    for (uint32_t r = rep_lo; r < rep_hi; ++r) {
        /* the end time is one rounded product of the cumulative horizon, so run(a); run(b) ends
         * exactly where run(a + b) ends */
        s->reps[r].H_total += horizon_iters;
        run_rep(s, r, (double)s->reps[r].H_total * tau_ref(s));
    }
    return 0;
}

/* Advance to the absolute time T (controllers that act at fixed epochs). */
int orc_run_until(orc_sim *s, double T, uint32_t rep_lo, uint32_t rep_hi)
{
    if (!s || rep_lo > rep_hi || rep_hi > s->cfg.R) return -1;
    for (uint32_t r = rep_lo; r < rep_hi; ++r) {
        if (T < s->reps[r].T_end) return -1;
        run_rep(s, r, T);
    }
    return 0;
}

/* New policy parameters from now on (online replanning, Section 6.2): nothing running is pre-empted, the new
 * split governs later placement and admission.  Single-block configurations only. */
int orc_set_targets(orc_sim *s, const orc_targets *tg)
{
    if (!s || !tg || s->cfg.nblk != 1 || tg->M > s->cfg.N) return -1;
    s->tg[0] = *tg;
    return 0;
}

int orc_reset_stats(orc_sim *s)
{
    if (!s) return -1;
    for (uint32_t r = 0; r < s->cfg.R; ++r) {
        rep_t *R = &s->reps[r];
        memset(&R->st, 0, sizeof R->st);
        R->T_reset = R->T_end;
        for (uint32_t i = 0; i < s->cfg.I; ++i) {
            area_t *as[5] = { &R->aQp[i], &R->aX[i], &R->aQd[i], &R->aYm[i], &R->aYs[i] };
            for (int k = 0; k < 5; ++k) { as[k]->area = 0.0; as[k]->t_last = R->T_end; }
        }
        if (R->h_ttft) {
            memset(R->h_ttft, 0, (size_t)s->cfg.I * ORC_NBIN * sizeof(uint64_t));
            memset(R->h_tpot, 0, (size_t)s->cfg.I * ORC_NBIN * sizeof(uint64_t));
        }
    }
    return 0;
}

int orc_stats(const orc_sim *s, orc_rep_stats *per_rep, uint64_t *hist_ttft, uint64_t *hist_tpot)
{
    if (!s || !per_rep) return -1;
    const orc_config *c = &s->cfg;
    for (uint32_t r = 0; r < c->R; ++r) {
        const rep_t *R = &s->reps[r];
        orc_rep_stats st = R->st;
        double T = R->T_end;
        st.T_elapsed = T - R->T_reset;
        for (uint32_t i = 0; i < c->I; ++i) {
            orc_class_stats *cs = &st.cls[i];
            uint32_t Qd = R->Qd_pool[0][i] + R->Qd_pool[1][i];
            cs->Qp = R->pq_n[i]; cs->X = R->X[i]; cs->Qd = Qd; cs->Ym = R->Ym[i]; cs->Ys = R->Ys[i];
            /* integrals are reported up to the end of the run without touching the stored state */
            cs->area_Qp = R->aQp[i].area + (double)R->pq_n[i] * (T - R->aQp[i].t_last);
            cs->area_X = R->aX[i].area + (double)R->X[i] * (T - R->aX[i].t_last);
            cs->area_Qd = R->aQd[i].area + (double)Qd * (T - R->aQd[i].t_last);
            cs->area_Ym = R->aYm[i].area + (double)R->Ym[i] * (T - R->aYm[i].t_last);
            cs->area_Ys = R->aYs[i].area + (double)R->Ys[i] * (T - R->aYs[i].t_last);
        }
        per_rep[r] = st;
        if (c->hist && hist_ttft && hist_tpot) {
            size_t n = (size_t)c->I * ORC_NBIN;
            memcpy(hist_ttft + (size_t)r * n, R->h_ttft, n * sizeof(uint64_t));
            memcpy(hist_tpot + (size_t)r * n, R->h_tpot, n * sizeof(uint64_t));
        }
    }
    return 0;
}

int orc_server_state(const orc_sim *s, uint32_t r, uint32_t *n_dec, uint32_t *it, double *t_next, uint32_t *pf_rem)
{
    if (!s || r >= s->cfg.R) return -1;
    const rep_t *R = &s->reps[r];
    for (uint32_t g = 0; g < s->cfg.N; ++g) {
        const server_t *v = &R->srv[g];
        if (n_dec) n_dec[g] = v->n_dec;
        if (it) it[g] = v->it;
        if (t_next) t_next[g] = v->running ? v->t_next : INFINITY;
        if (pf_rem) pf_rem[g] = v->pf_present ? v->pf_rem : 0;
    }
    return 0;
}

void orc_destroy(orc_sim *s)
{
    if (!s) return;
    for (uint32_t r = 0; r < s->cfg.R; ++r) {
        rep_t *R = &s->reps[r];
        for (uint32_t i = 0; i < s->cfg.I; ++i) free(R->pq[i]);
        for (uint32_t p = 0; p < 2; ++p) free(R->dq[p]);
        for (uint32_t g = 0; g < s->cfg.N; ++g) free(R->srv[g].slots);
        free(R->srv); free(R->h_ttft); free(R->h_tpot);
    }
    free(s->reps); free(s->rates); free(s->lengths); free(s->tg); free(s->inj_t); free(s->inj_job);
    free(s);
}
