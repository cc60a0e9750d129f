/*
 * CPU oracle of the many-replication gate-and-route simulation.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded, event-by-event reference: one replication at a time, a
 * linear scan over every event source per event, no batching, no look-ahead.  It exists so
 * that tests and the benchmark's CPU-baseline leg can check and time the GPU library against
 * an independent implementation.  It shares no source, header, table or helper with the CUDA
 * path; the product path never calls it.
 *
 * What it simulates (paper sections in brackets):
 *   - n = N GPUs, each with at most one prefill and at most B decode streams, prefill in chunks
 *     of C tokens, one iteration advances every active decode by one token and the prefill by
 *     one chunk                                                        [Sections 2.1, 2.2, 2.3]
 *   - iteration time from the two-regime law tau_solo / tau_mix(C)     [Eq. (1)-(3)], widened to
 *     six coefficients so that a per-decode and a per-KV-token slope can be switched on
 *   - Poisson arrivals of rate n*lambda_i, exponential patience theta_i in both queues, through
 *     the random time-change representation                              [Section 2.3, Eq. (7)-(9)]
 *   - static planning: GPUs 0..M-1 mixed, M..N-1 solo                   [Section 4.1]
 *   - prefill gate: occupancy deviation xi_i, or static D_i/P_i priority [Sections 4.1, 5.1.1]
 *   - decode router: solo-first with one FCFS buffer, or the SLI-aware
 *     randomized split with two buffers, optionally with class selection
 *     inside each pool by the weights varpi; or no router at all (decode on the
 *     GPU that prefilled, EC ablation study)                              [Sections 4.1, 5.2, EC general SLI extension]
 *   - revenue under bundled and separate charging                        [Eq. (21)-(23)]
 *   - piecewise-constant rate / target tables switched at block ends without pre-emption
 *                                                                        [Section 6.2, online controller]
 *
 * Parity pins: Philox against its published known-answer vectors; qlog against libm; the event
 * dynamics against hand-computed trajectories, flow-balance identities (Eq. (15)-(20)), capacity
 * constraints (Eq. (12)-(14)), a finite-horizon Little identity, a no-contention closed form and
 * convergence of revenue to the LP optimum; the KV-token bookkeeping of the KV slope and the role change of
 * a GPU at a block end against hand-computed trajectories and the request-by-request replay; the uniformity
 * of random placement and of the abandoning request by chi-square; broken copies of this file must fail
 * these pins (tests/test_oracle_kv_and_block_switch.py).  The trace-replay revenue tables the paper prints need
 * its production traces: parity unpinned for those numbers.
 */
#ifndef QSIM_ORACLE_H
#define QSIM_ORACLE_H

#include <stdint.h>
#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_MAXI 8
#define ORC_LMAX 8192
#define ORC_NBIN 1024

typedef struct {
    uint32_t I, N, R, B, C, nblk;
    uint32_t gate, router, placement, pricing, length_mode, qcap, hist, n_inject;
    uint64_t seed, rep_offset;
    double block_len;
} orc_config;

typedef struct {
    uint32_t P, D, prio_rank, pad;
    double theta;
} orc_class;

typedef struct {
    uint32_t M, pad;
    double xstar[ORC_MAXI], n_xstar[ORC_MAXI], n_qpstar[ORC_MAXI], p_solo[ORC_MAXI];
    double w_solo[ORC_MAXI], w_mix[ORC_MAXI];   /* varpi_s,i, varpi_m,i of the general SLI-aware router */
} orc_targets;

typedef struct {
    uint64_t arrivals, admitted, prefill_done, placed_mixed, placed_solo, done_mixed, done_solo;
    uint64_t abandoned_p, abandoned_d, overflow, overflow_d, tokens_in_prefilled, tokens_in_completed, tokens_out_completed;
    uint32_t Qp, X, Qd, Ym, Ys, pad;
    double area_Qp, area_X, area_Qd, area_Ym, area_Ys, sum_ttft, sum_tpot;
} orc_class_stats;

typedef struct {
    orc_class_stats cls[ORC_MAXI];
    uint64_t iters_mixed, iters_solo, events;
    double busy_mixed, busy_solo, T_elapsed;
} orc_rep_stats;

/* one line of the optional event trace */
enum { ORC_EV_ARRIVAL = 1, ORC_EV_ADMIT, ORC_EV_PREFILL_DONE, ORC_EV_PLACE, ORC_EV_DECODE_DONE,
       ORC_EV_ABANDON_P, ORC_EV_ABANDON_D, ORC_EV_ITER_END, ORC_EV_BLOCK, ORC_EV_OVERFLOW };
typedef struct {
    double t;         /* event time */
    double aux;       /* ITER_END: tau of the finished iteration; others: 0 */
    uint64_t job;     /* arrival ordinal of the job within its class (ITER_END/BLOCK: iteration / block index) */
    int32_t type, cls, server, rep;
} orc_trace_rec;

typedef struct orc_sim orc_sim;

/* All input arrays are copied.  lengths: NULL or [I][2][ORC_LMAX]; rates: [nblk][I];
 * inject_t/inject_job ([n_inject], [n_inject][3] = class,P,D): NULL unless cfg->n_inject > 0. */
int orc_create(orc_sim **out, const orc_config *cfg, const orc_class *classes, const double *rates,
               const uint32_t *lengths, const double *prices, const double *coeffs,
               const orc_targets *targets, const double *inject_t, const uint32_t *inject_job);
/* Optional trace sink; records beyond cap are counted but dropped. */
int orc_set_trace(orc_sim *s, orc_trace_rec *buf, uint64_t cap);
uint64_t orc_trace_count(const orc_sim *s);
/* Advance replications [rep_lo, rep_hi) by horizon_iters more iterations of horizon: the new end time is
 * (total horizon so far) * tau_ref, tau_ref = one full solo iteration. */
int orc_run(orc_sim *s, uint64_t horizon_iters, uint32_t rep_lo, uint32_t rep_hi);
int orc_run_until(orc_sim *s, double T, uint32_t rep_lo, uint32_t rep_hi);
int orc_set_targets(orc_sim *s, const orc_targets *tg);
int orc_reset_stats(orc_sim *s);
/* per_rep: [R]; hist_ttft / hist_tpot: NULL or uint64 [R][I][ORC_NBIN] */
int orc_stats(const orc_sim *s, orc_rep_stats *per_rep, uint64_t *hist_ttft, uint64_t *hist_tpot);
/* per-server snapshot of replication r: n_dec[N], it[N], t_next[N] (idle: +inf), pf_rem[N] */
int orc_server_state(const orc_sim *s, uint32_t r, uint32_t *n_dec, uint32_t *it, double *t_next, uint32_t *pf_rem);
void orc_destroy(orc_sim *s);

/* building blocks exposed so that tests can pin them one by one */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
double orc_qlog(double x);
double orc_u53(uint32_t w0, uint32_t w1);
double orc_tau(const double coeffs[6], uint32_t p, uint32_t d, uint64_t K);
uint32_t orc_table_length(const uint32_t *thr, uint32_t w);
uint32_t orc_hist_bin(double x);

#ifdef __cplusplus
}
#endif
#endif
