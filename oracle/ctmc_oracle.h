/*
 * CPU oracle of the exponential-service model of the gate-and-route network.  TEST INFRASTRUCTURE ONLY:
 * only tests, the smoke check and the benchmark's CPU legs may call it; the CUDA library shares nothing
 * with it.
 *
 * What it simulates: the stochastic model of Section 2.3 as the paper states it, not the iteration-level
 * simulator.  Per class i: Poisson arrivals of rate n lambda_i, exponential prefill service of rate
 * mu_p,i, exponential decode service of rate mu_m,i on a mixed GPU and mu_s,i on a solo GPU (Eq. (4)),
 * exponential patience theta_i in the prefill queue and in the decode buffer, all through the random
 * time-change representation of Eq. (7)-(9).  Policy: static planning with M mixed GPUs (Section 4.1),
 * the occupancy gate or the priority gate (Sections 4.1, 5.1.1), the solo-first router with one FCFS
 * buffer or the SLI-aware randomized router with one buffer per pool (Sections 4.1, 5.2).  Requests of a
 * class are exchangeable in this model, so the state is the vector (Q_p,i, X_i, Q_d,i, Y_m,i, Y_s,i) plus
 * the class order of the decode buffers; capacities are those of the static partition as the optimality
 * proof uses them: sum X <= M, sum Y_m <= M (B-1), sum Y_s <= (n-M) B.
 *
 * Parity pins (tests/test_ctmc_oracle.py): flow balance Eq. (15)-(20) and the capacity constraints on
 * every run; the M/M/infinity law of an uncontended stage; the stationary mean of the M/M/1+M prefill
 * queue from its birth-death balance equations; Poisson arrival counts; convergence of per-GPU revenue
 * to the LP optimum and of X_i/n to x*_i as n grows (the optimality theorems of Sections 4 and 5).
 */
#ifndef CTMC_ORACLE_H
#define CTMC_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    uint32_t I, N, M, B, R, qcap;
    uint32_t gate;     /* 0 occupancy, 1 priority */
    uint32_t router;   /* 0 solo-first, 1 SLI-aware randomized */
    uint64_t seed, rep_offset;
} ctmc_config;

typedef struct {
    double lambda, theta, mu_p, mu_m, mu_s;       /* per-GPU arrival rate; patience; service rates, Eq. (4) */
    double xstar, n_xstar, n_qpstar, p_solo;      /* LP targets x*_i, n x*_i, n q*_p,i and the routing probability p_s,i */
    uint32_t prio_rank, pad;
} ctmc_class;

enum { CTMC_ARRIVALS = 0, CTMC_ADMITTED, CTMC_PREFILL_DONE, CTMC_PLACED_MIXED, CTMC_PLACED_SOLO, CTMC_DONE_MIXED,
       CTMC_DONE_SOLO, CTMC_ABANDONED_P, CTMC_ABANDONED_D, CTMC_OVERFLOW_D, CTMC_NCOUNT };

typedef struct {
    uint64_t cnt[8][CTMC_NCOUNT];
    uint32_t state[8][5];      /* Q_p, X, Q_d, Y_m, Y_s at the end time */
    uint32_t pad[8];
    double area[8][5];         /* time integrals of the same five counts */
    uint64_t events;
    double T_elapsed;
} ctmc_rep_stats;

typedef struct ctmc_sim ctmc_sim;

int ctmc_create(ctmc_sim **out, const ctmc_config *cfg, const ctmc_class *classes);
int ctmc_run_until(ctmc_sim *s, double T_end, uint32_t rep_lo, uint32_t rep_hi);   /* events with t <= T_end */
int ctmc_stats(const ctmc_sim *s, ctmc_rep_stats *per_rep);                        /* [R] */
void ctmc_destroy(ctmc_sim *s);

#ifdef __cplusplus
}
#endif
#endif
