/*
 * qsim: many-replication simulation of a multiclass LLM-inference queueing network under the
 * gate-and-route policy, on one NVIDIA B200 (sm_100a).  C ABI; no C++ or framework types cross it.
 *
 * Model (paper sections in brackets).  A replication is a cluster of n = N GPUs.  Each GPU holds at
 * most one prefill and at most B decode streams; a prefill advances C tokens per iteration and every
 * active decode emits one token per iteration [Sections 2.1-2.2].  An iteration whose batch holds p
 * prefill tokens, d decodes and K resident KV tokens lasts
 *     tau = (p > 0 ? alpha_m + beta p + delta_m d : alpha_s + delta_s d) + kappa K,
 * which contains the paper's two regimes tau_mix(C) = alpha + beta C and tau_solo = c  [Eq. (1)-(3)]
 * and its solo fit with a KV slope [Section 6.1].  Class-i requests arrive as a Poisson process of
 * rate n lambda_i and wait with exponential patience theta_i in the prefill queue and in the decode
 * buffer [Section 2.3, Eq. (7)-(9)].  GPUs 0..M-1 are mixed (they keep one slot for prefill, so at most
 * B-1 decodes), GPUs M..N-1 are solo [Section 4.1, Static Planning].  The prefill gate admits the
 * waiting class with the smallest occupancy deviation (X_i - n x*_i)/x*_i, ties to the largest
 * Q_p,i - n q*_p,i [Section 4.1], or the class with the largest D_i/P_i [Section 5.1.1].  The decode
 * router serves one FCFS buffer, solo GPUs first [Section 4.1], or splits jobs between a solo and a
 * mixed buffer with probability p_s,i [Section 5.2], optionally picking the class inside each pool by
 * the weights varpi [EC, General SLI-aware Extension].  Rates and targets are piecewise constant over
 * blocks of block_len seconds and switch without pre-emption [Section 6.2].  Revenue is reported
 * under bundled and separate charging [Eq. (21)-(23)] from integer token counters.
 *
 * Determinism.  Random numbers are Philox4x32-10 with key = seed and counter =
 * (index, stream, replication); clocks are IEEE doubles, every operation rounded to nearest and never
 * contracted to FMA.  Integer results do not depend on the launch shape or on how replications are
 * split over handles (rep_offset).
 *
 * Pointers: every argument marked [host] is ordinary host memory owned by the caller and is copied
 * before the call returns; [device] is device memory owned by the caller that must stay valid until
 * qsim_destroy.  All functions return QSIM_OK (0) or a negative error; qsim_last_error() gives the
 * calling thread's last message.  A handle must not be used from two threads at once.
 */
#ifndef QSIM_H
#define QSIM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QSIM_MAXI 8       /* classes */
#define QSIM_LMAX 8192    /* largest request length; stride of the length tables */
#define QSIM_NBIN 1024    /* histogram bins: 32 per octave from 2^-20 s */

enum {
    QSIM_OK = 0,
    QSIM_EINVAL = -1,      /* bad argument or unsupported size */
    QSIM_ENOMEM = -2,      /* host or device allocation failed */
    QSIM_EWORKSPACE = -3,  /* workspace missing, too small or misaligned */
    QSIM_ECUDA = -4,       /* a CUDA call failed; the message names it */
    QSIM_EOVERFLOW = -5,   /* a replication hit an internal bound (message names replication and bound) */
    QSIM_ESTATE = -6       /* call out of order (run before bind, ...) */
};

enum { QSIM_GATE_OCCUPANCY = 0, QSIM_GATE_PRIORITY = 1,
       QSIM_GATE_FCFS = 2 /* oldest waiting request first: the FCFS-and-Route ablation of the paper's EC */ };
enum { QSIM_ROUTER_SOLO_FIRST = 0, QSIM_ROUTER_SLI = 1,
       QSIM_ROUTER_SLI_GENERAL = 2 /* two pools as QSIM_ROUTER_SLI; a freed slot goes to a class drawn with the pool's
                                      weights varpi among the classes that wait there, oldest request of the class
                                      first [EC, General SLI-aware Extension] */,
       QSIM_ROUTER_IMMEDIATE = 3   /* no router: a request decodes on the GPU that prefilled it, in the slot it holds
                                      (the "immediate same-slot decoding" ablations of the EC ablation study; with
                                      M = N it also drops the static partition) */ };
enum { QSIM_PLACE_RANDOM = 0, QSIM_PLACE_LEAST_LOADED = 1 };
enum { QSIM_PRICING_BUNDLED = 0, QSIM_PRICING_SEPARATE = 1 };
enum { QSIM_LENGTH_FIXED = 0, QSIM_LENGTH_TABLE = 1 };

typedef struct qsim qsim_t;

typedef struct {
    uint32_t size;         /* sizeof(qsim_config), checked */
    uint32_t I, N, R;      /* classes (<= 8), GPUs per replication (<= 4096), replications of this handle */
    uint32_t B, C;         /* decode cap per GPU (<= 4096), prefill chunk in tokens (<= 65535) */
    uint32_t nblk;         /* number of rate/target blocks (>= 1) */
    uint32_t gate, router, placement, pricing, length_mode;
    uint32_t qcap;         /* capacity, in requests, of each per-class prefill queue and each decode buffer */
    uint32_t hist;         /* 1: record TTFT / TPOT histograms */
    uint64_t seed;
    uint64_t rep_offset;   /* global index of this handle's replication 0 (sharding over handles / GPUs) */
    double block_len;      /* seconds; ignored when nblk == 1 */
} qsim_config;

typedef struct {
    uint32_t P, D;         /* prompt / output tokens of a class-i request when length_mode is FIXED (1..8192) */
    uint32_t prio_rank;    /* priority gate: smaller rank is served first */
    uint32_t reserved;
    double theta;          /* patience rate theta_i >= 0 (1/s); 0 disables abandonment */
} qsim_class;

typedef struct {           /* policy parameters of one block, from the steady-state LP (Eq. (36), (38)) */
    uint32_t M;            /* number of mixed GPUs, ceil(n sum_i x*_i) */
    uint32_t reserved;
    double xstar[QSIM_MAXI];     /* x*_i   (a class with x*_i = 0 is never admitted by the occupancy gate) */
    double n_xstar[QSIM_MAXI];   /* n x*_i */
    double n_qpstar[QSIM_MAXI];  /* n q*_p,i */
    double p_solo[QSIM_MAXI];    /* p_s,i of the SLI-aware router */
    double w_solo[QSIM_MAXI];    /* varpi_s,i >= 0: class-selection weights of the solo pool (QSIM_ROUTER_SLI_GENERAL only) */
    double w_mix[QSIM_MAXI];     /* varpi_m,i >= 0: the same for the mixed pool */
} qsim_targets;

typedef struct {
    /* cumulative counts since the last qsim_reset_stats: A, U_p, S_p, U_dm, U_ds, S_dm, S_ds, B_p, B_d */
    uint64_t arrivals, admitted, prefill_done, placed_mixed, placed_solo, done_mixed, done_solo;
    uint64_t abandoned_p, abandoned_d;
    uint64_t overflow, overflow_d;       /* requests dropped at a full prefill queue / decode buffer (0 when qcap fits) */
    uint64_t tokens_in_prefilled;        /* sum of P over finished prefills (separate charging credits c_p here) */
    uint64_t tokens_in_completed;        /* sum of P over finished requests (bundled charging credits c_p here) */
    uint64_t tokens_out_completed;       /* sum of D over finished requests */
    uint32_t Qp, X, Qd, Ym, Ys, reserved;  /* state at the end of the run; Ym / Ys by the group of the GPU at placement */
    double area_Qp, area_X, area_Qd, area_Ym, area_Ys;   /* time integrals of those counts */
    double sum_ttft, sum_tpot;           /* sums over finished prefills / finished requests */
} qsim_class_stats;

typedef struct {
    qsim_class_stats cls[QSIM_MAXI];
    uint64_t iters_mixed, iters_solo;    /* finished iterations with / without a prefill chunk */
    uint64_t events;                     /* arrivals + abandonments + block switches + iteration ends */
    double busy_mixed, busy_solo;        /* total duration of those iterations */
    double T_elapsed;                    /* simulated seconds since the last reset */
} qsim_rep_stats;

/*
 * Create a handle [Sections 2.3, 4.1: primitives and policy parameters].  [host] cfg, classes[I],
 * rates[nblk][I] (per-GPU lambda_i; the cluster rate is N lambda_i), lengths (NULL, or
 * [I][2][QSIM_LMAX] non-decreasing thresholds: a uniform 32-bit word w maps to length
 * 1 + #{j < QSIM_LMAX-1 : thr[j] <= w}; kind 0 = prompt, 1 = output), prices {c_p, c_d},
 * iter_time_coeffs {alpha_m, beta, delta_m, alpha_s, delta_s, kappa}, lp_targets[nblk].
 * Allocates a few hundred KB of device memory for the tables on the current device.
 */
int qsim_create(qsim_t **out, const qsim_config *cfg, const qsim_class *classes, const double *rates,
                const uint32_t *lengths, const double *prices, const double *iter_time_coeffs,
                const qsim_targets *lp_targets);

/* Bytes of device memory qsim_bind needs for this handle (state of all R replications). */
int qsim_workspace_bytes(const qsim_t *h, size_t *bytes);

/*
 * Give the handle its state memory: [device] workspace of at least qsim_workspace_bytes, 256-byte
 * aligned; cuda_stream is a cudaStream_t (NULL = default stream) on which every later launch and copy
 * of this handle is ordered.  Initialises all replications to the empty system at t = 0 (any converging
 * initial state is admissible, Assumption 1).
 */
int qsim_bind(qsim_t *h, void *dev_workspace, size_t bytes, void *cuda_stream);

/*
 * Checkpoint / resume.  All state of the replications lives in the caller's workspace, so a checkpoint is a copy of
 * its first qsim_workspace_bytes bytes taken between calls (after qsim_run / qsim_run_until has returned), and a
 * resume is: qsim_create with the same arguments, copy the bytes into a [device] workspace, then this call in place of
 * qsim_bind.  Nothing is initialised; the next qsim_run continues where the checkpointed run stopped, with the results
 * of an uninterrupted sequence of the same calls [the time horizon of Eq. (21)-(23) composes, see qsim_run].  Targets installed with
 * qsim_set_targets are part of the handle, not of the workspace: install them again.  QSIM_ESTATE if the bytes hold
 * no resumable state (some replication stopped on an internal error) or were saved by a handle of another configuration or
 * layout (a fingerprint of both is kept in the workspace).
 */
int qsim_bind_restore(qsim_t *h, void *dev_workspace, size_t bytes, void *cuda_stream);

/*
 * Advance every replication by horizon_iters more iterations of horizon [event-driven dynamics of
 * Section 2.3 under the policies of Sections 4-5]: the new end time is H * tau_ref, H the total horizon
 * requested so far and tau_ref = tau(0, B, 0) (one full solo iteration).  Events with time <= the new end
 * are processed.  Calls compose: run(a); run(b) leaves exactly the simulated state and the integer statistics of
 * run(a + b); the fp64 sums over finished requests (areas of Y_m and Y_s, TPOT sums) are added to the totals once per
 * launch in the warp-per-replication kernels, so there they agree up to the order of additions.  When the replications
 * outnumber the blocks the device holds at a time by a small factor, a call runs its horizon in several chunks per
 * replication inside one launch, with the result of as many successive calls (environment variable QSIM_CHUNKS=1
 * turns that off, QSIM_CHUNKS=K asks for K chunks).  QSIM_ECUDA if a block of such a launch gave up waiting for the
 * chunk before its own (the wait is bounded; the state is then unusable).
 * qsim_stats / qsim_sync wait for completion.
 */
int qsim_run(qsim_t *h, uint64_t horizon_iters);

/*
 * Advance every replication to the absolute simulated time T seconds (T not before the end of the previous
 * call); otherwise like qsim_run.  Meant for controllers that act at fixed epochs (online replanning every
 * 10 s, Section 6.2).  Do not mix with qsim_run on one handle: the two keep separate notions of the end time.
 */
int qsim_run_until(qsim_t *h, double T);

/*
 * Trace replay (Section 6.2): replace the Poisson source by a list of arrivals, the same for every
 * replication.  [host] t[n] ascending times in seconds, job[n][3] = {class, P, D}.  Call between qsim_create
 * and qsim_bind; needs nblk == 1.  The rates of qsim_create are then ignored.
 */
int qsim_set_injected(qsim_t *h, const double *t, const uint32_t *job, uint64_t n);

/*
 * Replace the policy parameters (M, x*, n x*, n q*_p, p_s) from now on, e.g. after re-solving the LP with
 * re-estimated rates (Eq. (45)-(46)).  Running service is not pre-empted; the new split governs later
 * placement and admission, exactly like a block switch.  Needs nblk == 1; takes effect at the next run call.
 */
int qsim_set_targets(qsim_t *h, const qsim_targets *lp_targets);

/* Upper bound on the rounds (one non-local event plus the iteration ends before it) one replication
 * processes per kernel launch (default 2^28); a replication that reaches it is continued by further
 * launches with identical results. */
int qsim_set_event_budget(qsim_t *h, uint64_t events_per_launch);

/* Wait until all work queued on the handle's stream has finished; reports sticky replication errors. */
int qsim_sync(qsim_t *h);

/*
 * Copy statistics [Eq. (15)-(23): cumulative flows, state, revenue counters] to [host] per_rep[R] (may
 * be NULL), totals (sums over replications taken in replication order; may be NULL), hist_ttft /
 * hist_tpot (uint64 [R][I][QSIM_NBIN]; may be NULL; zeros unless cfg.hist).  Bin of a latency x:
 * clamp((bits(x) >> 47) - ((1023 - 20) << 5), 0, QSIM_NBIN - 1).  Synchronises the stream.
 */
int qsim_stats(qsim_t *h, qsim_rep_stats *totals, qsim_rep_stats *per_rep, uint64_t *hist_ttft,
               uint64_t *hist_tpot);

/*
 * Latency percentiles over all replications from the histograms (cfg.hist must be 1): for each class i and each
 * quantile q[k] in (0, 1], ttft[i * nq + k] and tpot[i * nq + k] receive the lower edge, in seconds, of the first
 * histogram bin at which the cumulative count reaches ceil(q[k] * total); NaN for a class without samples.  Bins are
 * 32 per octave, so a percentile is exact to 2.2 % [the paper reports mean / P95 / P99 TTFT and TPOT, Section 6.2,
 * without defining an estimator].  [host] q[nq], ttft[I * nq], tpot[I * nq].  Synchronises the stream.
 */
int qsim_latency_percentiles(qsim_t *h, const double *q, uint32_t nq, double *ttft, double *tpot);

/* Zero all counters, integrals and histograms and restart T_elapsed; the simulated state is kept. */
int qsim_reset_stats(qsim_t *h);

/* Revenue per GPU per second since the last reset from totals [Eq. (22), (23)]:
 * (c_p tokens_in + c_d tokens_out) / (N sum_r T_elapsed). */
int qsim_revenue(const qsim_t *h, const qsim_rep_stats *totals, double *bundled_rate, double *separate_rate);

/* Per-GPU snapshot of replication r into [host] arrays of N entries (any may be NULL): decodes held,
 * finished iterations, end of the running iteration (+inf when idle), prefill tokens left. */
int qsim_server_state(qsim_t *h, uint32_t r, uint32_t *n_dec, uint32_t *it, double *t_next, uint32_t *pf_rem);

/*
 * One call from host buffers to host results: create, allocate the workspace with cudaMalloc, bind, run
 * horizon_iters, copy statistics back, free everything.  Arguments as in qsim_create / qsim_stats.
 */
int qsim_simulate(const qsim_config *cfg, const qsim_class *classes, const double *rates,
                  const uint32_t *lengths, const double *prices, const double *iter_time_coeffs,
                  const qsim_targets *lp_targets, uint64_t horizon_iters, qsim_rep_stats *totals,
                  qsim_rep_stats *per_rep);

/*
 * qsim_simulate for more replications than the device can hold at once [the convergence experiments of the EC run the
 * same instance for growing n; at n = 4096 GPUs with B = 256 one replication is tens of MB of state].  The R
 * replications are simulated `wave` at a time (0 = the largest wave that fits in nine tenths of the free device
 * memory), each wave from the empty system over horizon_iters, in one workspace that the call allocates once and
 * frees; random streams are keyed by the global replication index, so the result does not depend on `wave`: integer
 * statistics are identical and the totals are added in replication order.  [host] per_rep[R] and totals may be NULL;
 * waves_run (may be NULL) receives the number of waves.  Only whole runs can be split into waves: a handle that is
 * resumed by further qsim_run calls keeps all its replications resident.
 */
int qsim_simulate_waves(const qsim_config *cfg, const qsim_class *classes, const double *rates,
                        const uint32_t *lengths, const double *prices, const double *iter_time_coeffs,
                        const qsim_targets *lp_targets, uint64_t horizon_iters, uint32_t wave,
                        qsim_rep_stats *totals, qsim_rep_stats *per_rep, uint32_t *waves_run);

/*
 * The same simulation as qsim_simulate for callers that must not allocate.  (The paper has no
 * counterpart: this is a packaging variant of the library, not part of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plugin inside a serving process whose
 * own allocator has already reserved the whole card, so a fresh cudaMalloc would fail or evict; a
 * latency-critical section that cannot afford the device-wide synchronisation cudaMalloc / cudaFree
 * imply.  This entry point makes no device or pinned-memory allocation: no cudaMalloc, cudaFree or
 * cudaMallocHost (it does use the host heap for small temporaries, e.g. the index of the length tables).
 * All simulation state, the rate/target table and the length tables live in one array that is compiled
 * into the library: 32 MiB of device memory on every GPU that loads libqsim.so, held until the process exits.
 *
 * Arguments as in qsim_simulate ([host] inputs, [host] totals / per_rep[R] outputs, either may be NULL),
 * plus cuda_stream (a cudaStream_t, NULL = default stream) on which the copies and kernels are ordered;
 * the call returns after the stream has finished.  Histograms are not recorded (cfg.hist is ignored) and
 * nblk must be <= 64.  If the problem needs more than the 32 MiB (state grows with R, N*B and qcap) the
 * call fails with QSIM_EWORKSPACE and a message that states the bytes needed.
 *
 * The first call on each device looks up the array's device address; make that first call with the
 * device current and outside any stream capture.  Every call on a device shares the one array: calls
 * must not overlap on the GPU (two host threads, or two streams) or they corrupt each other.  Nothing
 * needs clearing by the caller - each call re-initialises the state it uses.
 */
int qsim_simulate_static(const qsim_config *cfg, const qsim_class *classes, const double *rates,
                         const uint32_t *lengths, const double *prices, const double *iter_time_coeffs,
                         const qsim_targets *lp_targets, uint64_t horizon_iters, qsim_rep_stats *totals,
                         qsim_rep_stats *per_rep, void *cuda_stream);

/*
 * Environment variables (diagnostics and cross-checks; none of them changes a result beyond the order of fp64 additions,
 * which the tests use): QSIM_FAMILY=warp|lane picks the kernel family (a warp, or a few warps, per replication; one
 * thread per replication) where the configuration allows both; QSIM_WARPS=1..16 the warps per replication of the first;
 * QSIM_LANE_LSH=2..5 the binary logarithm of the replications per warp of the second; QSIM_KERNEL=generic the kernel
 * instance that reads every feature from its parameters; QSIM_CHUNKS, see qsim_run.  Read when a handle is created
 * (QSIM_CHUNKS: at every qsim_run).
 */

/* Diagnostic: look-ahead rounds executed since the last reset, summed over replications (a round handles at
 * most one non-local event and every local iteration end before it).  Synchronises the stream. */
int qsim_round_count(qsim_t *h, uint64_t *rounds);

/* Diagnostic: out[0] = bytes per replication that qsim_stats copies to the host, out[1] = bytes of per-GPU
 * state staged per replication at kernel entry and exit, out[2] = shared memory per block, out[3] = warps per
 * replication. */
int qsim_layout_info(const qsim_t *h, uint64_t out[4]);

/* Kernel launches issued by this handle so far (for accounting in benchmarks). */
int qsim_launch_count(const qsim_t *h, uint64_t *launches);

/*
 * Exponential-service model [Section 2.3].  The paper's analysis models prefill, mixed decode and solo decode
 * service times as independent exponentials with the rates of Eq. (4), mu_p,i = C/(P_i tau), mu_m,i = 1/(D_i tau),
 * mu_s,i = gamma/D_i; arrivals are Poisson of rate n lambda_i and waiting requests have exponential patience
 * theta_i in the prefill queue and in the decode buffer, all driven by unit-rate Poisson processes on the
 * integrated intensities of Eq. (7)-(9).  The policy is the static partition with M mixed GPUs, the occupancy or
 * priority gate and the solo-first or SLI-aware router [Sections 4.1, 5.1.1, 5.2].  Requests of a class are
 * exchangeable, so a replication's state is (Q_p,i, X_i, Q_d,i, Y_m,i, Y_s,i) and the class order of the decode
 * buffers, with the capacities the optimality proof uses: sum_i X_i <= M, sum_i Y_m,i <= M (B-1),
 * sum_i Y_s,i <= (N-M) B.  These entry points keep no handle: the caller's device workspace holds all state.
 */
typedef struct {
    uint32_t size;             /* sizeof(qsim_ctmc_config) */
    uint32_t I, N, M, B, R;    /* classes, GPUs, mixed GPUs, decode cap per GPU, replications */
    uint32_t qcap;             /* capacity (requests) of each decode buffer; a finished prefill that finds it full is dropped and counted */
    uint32_t gate;             /* QSIM_GATE_OCCUPANCY or QSIM_GATE_PRIORITY */
    uint32_t router;           /* QSIM_ROUTER_SOLO_FIRST or QSIM_ROUTER_SLI */
    uint32_t reserved;
    uint64_t seed, rep_offset; /* Philox key; global index of replication 0 */
} qsim_ctmc_config;

typedef struct {
    double lambda, theta;                       /* per-GPU arrival rate, patience rate */
    double mu_p, mu_m, mu_s;                    /* Eq. (4) */
    double xstar, n_xstar, n_qpstar, p_solo;    /* x*_i, n x*_i, n q*_p,i, p_s,i as in qsim_targets */
    uint32_t prio_rank, reserved;               /* 0 = admitted first by QSIM_GATE_PRIORITY */
} qsim_ctmc_class;

typedef struct {
    /* per class: A, U_p, S_p, U_dm, U_ds, S_dm, S_ds, B_p, B_d, finished prefills dropped at a full buffer */
    uint64_t cnt[QSIM_MAXI][10];
    uint32_t state[QSIM_MAXI][5];   /* Q_p, X, Q_d, Y_m, Y_s at the end time */
    uint32_t reserved[QSIM_MAXI];
    double area[QSIM_MAXI][5];      /* time integrals of the same five counts over [0, T_elapsed] */
    uint64_t events;                /* jumps processed */
    double T_elapsed;               /* end time reached */
} qsim_ctmc_rep_stats;

/* Bytes of device memory the three calls below need for this configuration. */
int qsim_ctmc_workspace_bytes(const qsim_ctmc_config *cfg, size_t *bytes);

/* Empty system at t = 0 in [device] dev_workspace (256-byte aligned, at least qsim_ctmc_workspace_bytes; owned by
 * the caller); [host] cfg, classes[I].  One asynchronous launch on cuda_stream (a cudaStream_t, NULL = default). */
int qsim_ctmc_init(const qsim_ctmc_config *cfg, const qsim_ctmc_class *classes, void *dev_workspace, size_t bytes,
                   void *cuda_stream);

/* Process every jump with t <= T_end (seconds; T_end must not decrease between calls) in all R replications,
 * with the same cfg and classes as qsim_ctmc_init.  Returns after the stream has finished; launches (may be NULL)
 * receives the number of kernel launches it took. */
int qsim_ctmc_run_until(const qsim_ctmc_config *cfg, const qsim_ctmc_class *classes, void *dev_workspace, size_t bytes,
                        void *cuda_stream, double T_end, uint64_t *launches);

/* Copy the statistics of all replications to [host] per_rep[R]; time integrals are closed at the end time.
 * Synchronises the stream.  QSIM_EOVERFLOW if a replication stopped on an internal error. */
int qsim_ctmc_stats(const qsim_ctmc_config *cfg, const void *dev_workspace, size_t bytes, void *cuda_stream,
                    qsim_ctmc_rep_stats *per_rep);

/* Revenue per GPU per second of every replication of the exponential-service model from its counters [Eq. (21)-(23)]:
 * bundled charging credits c_p P_i + c_d D_i when a request finishes decoding; separate charging (separate != 0) credits
 * c_p P_i when its prefill finishes and c_d D_i when its decode finishes.  [host] per_rep[R] as filled by qsim_ctmc_stats,
 * P[I], D[I] mean prompt / output tokens, prices {c_p, c_d}; rate[R] receives revenue / (N T_elapsed). */
int qsim_ctmc_revenue(const qsim_ctmc_config *cfg, const qsim_ctmc_rep_stats *per_rep, const double *P, const double *D,
                      const double *prices, int separate, double *rate);

int qsim_destroy(qsim_t *h);

const char *qsim_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
