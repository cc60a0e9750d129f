/*
 * CPU oracle of the exponential-service (Markov chain) model of the gate-and-route network.
 * TEST INFRASTRUCTURE ONLY: see ctmc_oracle.h.  Compile with -ffp-contract=off.
 *
 * The model is Section 2.3 written out: for every class i seven unit-rate Poisson processes
 * (arrivals, abandonment from the prefill queue, abandonment from each decode buffer, prefill
 * completions, mixed and solo decode completions) run on the integrated intensities of Eq. (7)-(9).
 * A process with intensity c * n(t) keeps acc = integral of c n since its last jump and the exponential
 * level lvl of its next jump; its next jump time is recomputed whenever n changes.  One event at a
 * time, a linear scan over all processes per event.
 */
#include "ctmc_oracle.h"
#include "qsim_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

enum { K_ARR = 0, K_ABP = 1, K_ABD0 = 2, K_ABD1 = 3, K_SP = 4, K_SDM = 5, K_SDS = 6, NK = 7 };
/* Philox stream purposes (stream = purpose << 8 | class); 0..3 as in the iteration-level simulator */
static const uint32_t PURPOSE[NK] = { 0, 1, 2, 3, 8, 9, 10 };
enum { PURPOSE_SLI = 5 };

typedef struct { double acc, lvl, t_last, t_fire; uint64_t m; } clk_t;
typedef struct { double area, t_last; } area_t;

typedef struct {
    double t, T_end;
    clk_t clk[NK][ORC_MAXI];
    uint32_t Qp[ORC_MAXI], X[ORC_MAXI], Qd[2][ORC_MAXI], Ym[ORC_MAXI], Ys[ORC_MAXI];
    uint64_t sli_ord[ORC_MAXI];
    area_t aQp[ORC_MAXI], aX[ORC_MAXI], aQd[ORC_MAXI], aYm[ORC_MAXI], aYs[ORC_MAXI];
    uint64_t cnt[ORC_MAXI][CTMC_NCOUNT];
    uint64_t events;
    uint8_t *ring[2];
    uint32_t head[2], n[2];
    int err;
} rep_t;

struct ctmc_sim {
    ctmc_config cfg;
    ctmc_class cls[ORC_MAXI];
    rep_t *reps;
};

static void draw(const ctmc_sim *s, uint32_t r, uint32_t stream, uint64_t index, uint32_t w[4])
{
    uint32_t ctr[4] = { (uint32_t)index, (uint32_t)(index >> 32), stream, (uint32_t)(s->cfg.rep_offset + r) };
    uint32_t key[2] = { (uint32_t)s->cfg.seed, (uint32_t)(s->cfg.seed >> 32) };
    orc_philox4x32_10(ctr, key, w);
}

static double unit_exp(const ctmc_sim *s, uint32_t r, uint32_t k, uint32_t i, uint64_t m, uint32_t w[4])
{
    draw(s, r, (PURPOSE[k] << 8) | i, m, w);
    return -orc_qlog(orc_u53(w[0], w[1]));
}

/* intensity coefficient of process k of class i (per unit of the count it runs on) */
static double coef(const ctmc_sim *s, uint32_t k, uint32_t i)
{
    switch (k) {
    case K_ABP: case K_ABD0: case K_ABD1: return s->cls[i].theta;
    case K_SP: return s->cls[i].mu_p;
    case K_SDM: return s->cls[i].mu_m;
    case K_SDS: return s->cls[i].mu_s;
    default: return 0.0;
    }
}

static void area_touch(area_t *a, uint32_t count, double t)
{
    a->area = a->area + (double)count * (t - a->t_last);
    a->t_last = t;
}

/* the count that process k of class i runs on changes from n_old to n_new at time t */
static void clk_change(const ctmc_sim *s, rep_t *R, uint32_t k, uint32_t i, uint32_t n_old, uint32_t n_new, double t)
{
    const double c = coef(s, k, i);
    if (!(c > 0.0)) return;
    clk_t *q = &R->clk[k][i];
    q->acc = q->acc + (c * (double)n_old) * (t - q->t_last);
    q->t_last = t;
    if (n_new > 0) {
        double rem = q->lvl - q->acc;
        if (rem < 0.0) rem = 0.0;
        q->t_fire = t + rem / (c * (double)n_new);
    } else {
        q->t_fire = INFINITY;
    }
}

/* process k of class i has just jumped at time t and its count is now n_new: new level */
static void clk_fired(const ctmc_sim *s, rep_t *R, uint32_t r, uint32_t k, uint32_t i, uint32_t n_new, double t, uint32_t w[4])
{
    clk_t *q = &R->clk[k][i];
    const double c = coef(s, k, i);
    q->lvl = unit_exp(s, r, k, i, q->m, w);
    q->m += 1;
    q->acc = 0.0;
    q->t_last = t;
    q->t_fire = n_new > 0 ? t + q->lvl / (c * (double)n_new) : INFINITY;
}

static uint32_t total(const uint32_t *v, uint32_t I)
{
    uint32_t s = 0;
    for (uint32_t i = 0; i < I; ++i) s += v[i];
    return s;
}

/* setters that keep the time integrals and the clocks that run on the count in step */
static void set_Qp(const ctmc_sim *s, rep_t *R, uint32_t i, uint32_t v, double t)
{
    clk_change(s, R, K_ABP, i, R->Qp[i], v, t);
    area_touch(&R->aQp[i], R->Qp[i], t);
    R->Qp[i] = v;
}
static void set_X(const ctmc_sim *s, rep_t *R, uint32_t i, uint32_t v, double t)
{
    clk_change(s, R, K_SP, i, R->X[i], v, t);
    area_touch(&R->aX[i], R->X[i], t);
    R->X[i] = v;
}
static void set_Qd(const ctmc_sim *s, rep_t *R, uint32_t pool, uint32_t i, uint32_t v, double t)
{
    clk_change(s, R, pool ? K_ABD1 : K_ABD0, i, R->Qd[pool][i], v, t);
    area_touch(&R->aQd[i], R->Qd[0][i] + R->Qd[1][i], t);
    R->Qd[pool][i] = v;
}
static void set_Ym(const ctmc_sim *s, rep_t *R, uint32_t i, uint32_t v, double t)
{
    clk_change(s, R, K_SDM, i, R->Ym[i], v, t);
    area_touch(&R->aYm[i], R->Ym[i], t);
    R->Ym[i] = v;
}
static void set_Ys(const ctmc_sim *s, rep_t *R, uint32_t i, uint32_t v, double t)
{
    clk_change(s, R, K_SDS, i, R->Ys[i], v, t);
    area_touch(&R->aYs[i], R->Ys[i], t);
    R->Ys[i] = v;
}

/* prefill gate (Section 4.1 occupancy rule / Section 5.1.1 priority rule); -1 when no class may enter */
static int gate_class(const ctmc_sim *s, const rep_t *R)
{
    const ctmc_config *c = &s->cfg;
    int best = -1;
    if (c->gate == 1) {
        for (uint32_t i = 0; i < c->I; ++i)
            if (R->Qp[i] > 0 && (best < 0 || s->cls[i].prio_rank < s->cls[best].prio_rank)) best = (int)i;
        return best;
    }
    double bxi = 0.0, bdq = 0.0;
    for (uint32_t i = 0; i < c->I; ++i) {
        if (R->Qp[i] == 0 || !(s->cls[i].xstar > 0.0)) continue;
        const double xi = ((double)R->X[i] - s->cls[i].n_xstar) / s->cls[i].xstar;
        const double dq = (double)R->Qp[i] - s->cls[i].n_qpstar;
        if (best < 0 || xi < bxi || (xi == bxi && dq > bdq)) { best = (int)i; bxi = xi; bdq = dq; }
    }
    return best;
}

/* after every event: buffered decodes into free slots (solo group first), then the gate */
static void dispatch(const ctmc_sim *s, rep_t *R, double t)
{
    const ctmc_config *c = &s->cfg;
    const uint32_t cap_s = (c->N - c->M) * c->B, cap_m = c->M * (c->B - 1);
    const uint32_t npools = c->router == 1 ? 2u : 1u;
    for (uint32_t pool = 0; pool < npools; ++pool) {
        while (R->n[pool] > 0) {
            int to_solo;
            if (c->router == 1) {
                to_solo = pool == 0;
                if (to_solo ? total(R->Ys, c->I) >= cap_s : total(R->Ym, c->I) >= cap_m) break;
            } else {
                if (total(R->Ys, c->I) < cap_s) to_solo = 1;
                else if (total(R->Ym, c->I) < cap_m) to_solo = 0;
                else break;
            }
            const uint32_t i = R->ring[pool][R->head[pool]];
            R->head[pool] = (R->head[pool] + 1) % c->qcap;
            R->n[pool] -= 1;
            set_Qd(s, R, pool, i, R->Qd[pool][i] - 1, t);
            if (to_solo) { set_Ys(s, R, i, R->Ys[i] + 1, t); R->cnt[i][CTMC_PLACED_SOLO]++; }
            else         { set_Ym(s, R, i, R->Ym[i] + 1, t); R->cnt[i][CTMC_PLACED_MIXED]++; }
        }
    }
    while (total(R->X, c->I) < c->M) {
        const int i = gate_class(s, R);
        if (i < 0) break;
        set_Qp(s, R, (uint32_t)i, R->Qp[i] - 1, t);
        set_X(s, R, (uint32_t)i, R->X[i] + 1, t);
        R->cnt[i][CTMC_ADMITTED]++;
    }
    /* capacity constraints, Eq. (12)-(14) under the static partition */
    if (total(R->X, c->I) > c->M || total(R->Ym, c->I) > cap_m || total(R->Ys, c->I) > cap_s) R->err = 2;
}

static void init_rep(const ctmc_sim *s, uint32_t r)
{
    rep_t *R = &s->reps[r];
    uint32_t w[4];
    for (uint32_t i = 0; i < s->cfg.I; ++i) {
        for (uint32_t k = 0; k < NK; ++k) {
            clk_t *q = &R->clk[k][i];
            q->acc = 0.0; q->t_last = 0.0; q->t_fire = INFINITY;
            q->lvl = unit_exp(s, r, k, i, 0, w);
            q->m = 1;
        }
        const double Lam = (double)s->cfg.N * s->cls[i].lambda;
        if (Lam > 0.0) R->clk[K_ARR][i].t_fire = 0.0 + R->clk[K_ARR][i].lvl / Lam;
    }
}

static void run_rep(ctmc_sim *s, uint32_t r, double T_end)
{
    rep_t *R = &s->reps[r];
    const ctmc_config *c = &s->cfg;
    uint32_t w[4];
    R->T_end = T_end;
    while (!R->err) {
        /* earliest process; ties by process kind, then class */
        double te = INFINITY;
        uint32_t bk = 0, bi = 0;
        for (uint32_t k = 0; k < NK; ++k)
            for (uint32_t i = 0; i < c->I; ++i)
                if (R->clk[k][i].t_fire < te) { te = R->clk[k][i].t_fire; bk = k; bi = i; }
        if (!(te <= T_end)) break;
        const double t = te;
        R->t = t;
        R->events++;
        const uint32_t i = bi;
        switch (bk) {
        case K_ARR: {
            R->cnt[i][CTMC_ARRIVALS]++;
            set_Qp(s, R, i, R->Qp[i] + 1, t);
            clk_t *q = &R->clk[K_ARR][i];
            q->lvl = unit_exp(s, r, K_ARR, i, q->m, w);
            q->m += 1;
            q->t_fire = t + q->lvl / ((double)c->N * s->cls[i].lambda);
            break;
        }
        case K_ABP: {
            /* all waiting requests of a class are alike here, so the count alone changes */
            area_touch(&R->aQp[i], R->Qp[i], t);
            R->Qp[i] -= 1;
            R->cnt[i][CTMC_ABANDONED_P]++;
            clk_fired(s, R, r, K_ABP, i, R->Qp[i], t, w);
            break;
        }
        case K_ABD0: case K_ABD1: {
            const uint32_t pool = bk == K_ABD1;
            const uint32_t Q = R->Qd[pool][i];
            clk_fired(s, R, r, bk, i, Q - 1, t, w);
            /* a uniformly chosen waiting class-i request leaves the pool's FCFS buffer */
            uint32_t rank = (uint32_t)(((uint64_t)w[2] * Q) >> 32), pos = 0;
            for (pos = 0; pos < R->n[pool]; ++pos) {
                if (R->ring[pool][(R->head[pool] + pos) % c->qcap] != i) continue;
                if (rank == 0) break;
                --rank;
            }
            if (pos >= R->n[pool]) { R->err = 3; break; }
            for (uint32_t k = pos; k + 1 < R->n[pool]; ++k)
                R->ring[pool][(R->head[pool] + k) % c->qcap] = R->ring[pool][(R->head[pool] + k + 1) % c->qcap];
            R->n[pool] -= 1;
            area_touch(&R->aQd[i], R->Qd[0][i] + R->Qd[1][i], t);
            R->Qd[pool][i] = Q - 1;
            R->cnt[i][CTMC_ABANDONED_D]++;
            break;
        }
        case K_SP: {
            area_touch(&R->aX[i], R->X[i], t);
            R->X[i] -= 1;
            R->cnt[i][CTMC_PREFILL_DONE]++;
            clk_fired(s, R, r, K_SP, i, R->X[i], t, w);
            uint32_t pool = 0;
            if (c->router == 1) {
                /* SLI-aware router: one uniform per finished prefill decides the pool (Section 5.2) */
                draw(s, r, (PURPOSE_SLI << 8) | i, R->sli_ord[i]++, w);
                pool = orc_u53(w[0], w[1]) <= s->cls[i].p_solo ? 0u : 1u;
            }
            if (R->n[pool] >= c->qcap) {
                R->cnt[i][CTMC_OVERFLOW_D]++;
            } else {
                R->ring[pool][(R->head[pool] + R->n[pool]) % c->qcap] = (uint8_t)i;
                R->n[pool] += 1;
                set_Qd(s, R, pool, i, R->Qd[pool][i] + 1, t);
            }
            break;
        }
        case K_SDM: {
            area_touch(&R->aYm[i], R->Ym[i], t);
            R->Ym[i] -= 1;
            R->cnt[i][CTMC_DONE_MIXED]++;
            clk_fired(s, R, r, K_SDM, i, R->Ym[i], t, w);
            break;
        }
        default: {
            area_touch(&R->aYs[i], R->Ys[i], t);
            R->Ys[i] -= 1;
            R->cnt[i][CTMC_DONE_SOLO]++;
            clk_fired(s, R, r, K_SDS, i, R->Ys[i], t, w);
            break;
        }
        }
        if (R->err) break;
        dispatch(s, R, t);
    }
}

int ctmc_create(ctmc_sim **out, const ctmc_config *cfg, const ctmc_class *classes)
{
    if (!out || !cfg || !classes) return -1;
    if (cfg->I < 1 || cfg->I > ORC_MAXI || cfg->N < 1 || cfg->M > cfg->N || cfg->B < 1 || cfg->R < 1 || cfg->qcap < 1 ||
        cfg->gate > 1 || cfg->router > 1)
        return -1;
    ctmc_sim *s = (ctmc_sim *)calloc(1, sizeof *s);
    if (!s) return -2;
    s->cfg = *cfg;
    memcpy(s->cls, classes, cfg->I * sizeof(ctmc_class));
    s->reps = (rep_t *)calloc(cfg->R, sizeof(rep_t));
    if (!s->reps) { free(s); return -2; }
    for (uint32_t r = 0; r < cfg->R; ++r) {
        for (int p = 0; p < 2; ++p) {
            s->reps[r].ring[p] = (uint8_t *)calloc(cfg->qcap, 1);
            if (!s->reps[r].ring[p]) { ctmc_destroy(s); return -2; }
        }
        init_rep(s, r);
    }
    *out = s;
    return 0;
}

int ctmc_run_until(ctmc_sim *s, double T_end, uint32_t rep_lo, uint32_t rep_hi)
{
    if (!s || rep_hi > s->cfg.R) return -1;
    for (uint32_t r = rep_lo; r < rep_hi; ++r) {
        run_rep(s, r, T_end);
        if (s->reps[r].err) return -10 - s->reps[r].err;
    }
    return 0;
}

int ctmc_stats(const ctmc_sim *s, ctmc_rep_stats *per_rep)
{
    if (!s || !per_rep) return -1;
    for (uint32_t r = 0; r < s->cfg.R; ++r) {
        const rep_t *R = &s->reps[r];
        ctmc_rep_stats *o = &per_rep[r];
        memset(o, 0, sizeof *o);
        const double T = R->T_end;
        for (uint32_t i = 0; i < s->cfg.I; ++i) {
            memcpy(o->cnt[i], R->cnt[i], sizeof R->cnt[i]);
            o->state[i][0] = R->Qp[i]; o->state[i][1] = R->X[i]; o->state[i][2] = R->Qd[0][i] + R->Qd[1][i];
            o->state[i][3] = R->Ym[i]; o->state[i][4] = R->Ys[i];
            o->area[i][0] = R->aQp[i].area + (double)R->Qp[i] * (T - R->aQp[i].t_last);
            o->area[i][1] = R->aX[i].area + (double)R->X[i] * (T - R->aX[i].t_last);
            o->area[i][2] = R->aQd[i].area + (double)(R->Qd[0][i] + R->Qd[1][i]) * (T - R->aQd[i].t_last);
            o->area[i][3] = R->aYm[i].area + (double)R->Ym[i] * (T - R->aYm[i].t_last);
            o->area[i][4] = R->aYs[i].area + (double)R->Ys[i] * (T - R->aYs[i].t_last);
        }
        o->events = R->events;
        o->T_elapsed = T;
    }
    return 0;
}

void ctmc_destroy(ctmc_sim *s)
{
    if (!s) return;
    if (s->reps)
        for (uint32_t r = 0; r < s->cfg.R; ++r) { free(s->reps[r].ring[0]); free(s->reps[r].ring[1]); }
    free(s->reps);
    free(s);
}
