// Device side of qsim: one warp simulates one replication.
//
// Look-ahead.  The end of an iteration on a simulated GPU touches nothing outside that GPU unless a request
// finishes its prefill there (it must be routed, and the gate admits the next one) or a decode ends while
// requests wait in a decode buffer (the freed slot must be refilled).  All other iteration ends are
// "local".  A request placed on a running GPU only joins at that GPU's next iteration boundary, and no
// iteration is shorter than tau_min = min(alpha_m, alpha_s).  So in every round the warp finds the next
// non-local event (time T_int) and the earliest running iteration end T_min, and every lane finishes, in
// parallel, the local iteration ends of its own GPUs that come before min(T_int, T_min + tau_min, T_end):
// each GPU has at most one such end, and nothing that happens in that window can change another GPU's
// batch.  Decode completions found on the way are then retired by the whole warp, GPU by GPU, and only
// after that is the non-local event handled by the warp-wide path.  The outcome is event for event that of
// the one-at-a-time order; only the order in which some sums are accumulated differs.
//
// Ownership inside the warp (no two lanes ever write the same word, so the only synchronisation is a
// few __syncwarp per event):
//   * lane i (< I) owns class i: its arrival clock, prefill queue cursor, abandonment clocks, counts,
//     time integrals and statistics (struct ClassState, in shared memory);
//   * lane l owns GPUs l, l+32, l+64, ...: their clocks and batch state (structure-of-arrays in shared
//     memory, staged from / to global memory at kernel entry / exit);
//   * scalars every lane needs (event time, block, buffer cursors, ordinals) are kept replicated in
//     registers and updated identically by all lanes.
// The next event is a warp-wide argmin over every lane's earliest source (three redux.sync on the bit
// pattern of the positive doubles plus the source id, which encodes the tie order).  Decisions that look
// at all GPUs (least-loaded / k-th eligible GPU) are evaluated by the owners and reduced the same way.
//
// All clock arithmetic is IEEE double, one rounding per operation, never contracted (the file is also
// compiled with --fmad=false).
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace qsimdev {

constexpr int MAXI = 8;
constexpr int LMAX = 8192;
constexpr int NBIN = 1024;
constexpr unsigned FULL = 0xffffffffu;
constexpr uint32_t NONE32 = 0xffffffffu;
constexpr int TOUCH_CAP = 48;

// Compile-time specialisation of the run kernel.  With F_GENERIC every mode is read from the parameters at
// run time; otherwise the set bits say which features the instance contains and everything else is
// compiled out.  SPL > 0 fixes the number of simulated GPUs per lane (N <= 32 SPL) so the per-GPU loops unroll.
constexpr uint32_t F_GENERIC = 1, F_ABANDON = 2, F_SLI = 4, F_KAPPA = 8, F_HIST = 16, F_BLOCKS = 32, F_RANDOM = 64,
                   F_OCC = 128, F_SLOTS = 256, F_MW = 512, F_FCFS = 1024, F_SLIG = 2048, F_IMM = 4096;
// F_MW: several warps per replication.  Warp 0 (the master) runs the round loop and every event handler; the
// other warps (helpers) wait at a block barrier for commands and take their share of the per-GPU work of a
// round: rows r = warp, warp + W, ... of the candidate scan and of the local iteration ends / retirements.
enum { MW_SCAN = 1, MW_ENDS = 2, MW_EXIT = 3 };
struct MwCmd { unsigned long long lim_t; uint32_t op, lim_s, buffered, M, force, pad; };
struct MwRes { unsigned long long bt, tmin; uint32_t bs, progressed; };
constexpr int MW_MAX = 16;

// source ids: smaller id wins an exact tie in time
constexpr uint32_t SRC_BLOCK = 0, SRC_ARRIVAL = 1, SRC_ABP = 9, SRC_ABD0 = 17, SRC_ABD1 = 25, SRC_SERVER = 33;

enum { STREAM_ARRIVAL = 0, STREAM_ABANDON_P = 1, STREAM_ABANDON_D0 = 2, STREAM_ABANDON_D1 = 3,
       STREAM_PLACEMENT = 4, STREAM_SLI = 5, STREAM_SELECT0 = 6, STREAM_SELECT1 = 7 };
enum { WANT_SOLO = 0, WANT_MIX = 1, WANT_PREFILL = 2 };
enum { ERR_NONE = 0, ERR_INTERNAL = 1 };

struct AbClock { double acc, lvl, t_last, t_ab; unsigned long long m; };
struct Area { double area, t_last; };

struct ClassState {
    double ta;
    unsigned long long adraw, sli_ord;
    uint32_t ablk, nextP, nextD, pq_head, pq_n, X, Ym, Ys, Qd0, Qd1, pq_tail, pq_pad;   // pq_tail: one-thread-per-replication kernels
    AbClock abp, abd0, abd1;
    Area aQp, aX, aQd;
    double sYm_in, sYm_out, sYs_in, sYs_out;   // sums of (placement / completion time - T_reset): integral of Y = out - in + Y (T - T_reset)
    unsigned long long arrivals, admitted, prefill_done, placed_mixed, placed_solo, done_mixed, done_solo,
        abandoned_p, abandoned_d, overflow, overflow_d, tok_in_pf, tok_in_done, tok_out_done;
    double sum_ttft, sum_tpot;
};

struct RepHeader {
    double T_end, T_reset;
    unsigned long long place_ord, events, H_total, rounds;
    uint32_t blk, done, err, force;    // force: the next event must be followed by a dispatch (targets were replaced)
    double t_now;                      // time of the last event handled (one-thread-per-replication kernels)
    uint32_t seq, chunks_left;         // launches that split the horizon into chunks: hand-over stamp of the last chunk done, chunks not started yet
    uint32_t dq_head0, dq_head1, dq_n0, dq_n1;
    unsigned long long sel_ord0, sel_ord1;   // class selections drawn so far in the solo / mixed pool (general SLI router)
    unsigned long long iters_mixed[32], iters_solo[32];
    double busy_mixed[32], busy_solo[32];
    ClassState cs[MAXI];
};

static_assert(sizeof(ClassState) % 8 == 0 && (sizeof(ClassState) * MAXI) % 16 == 0, "ClassState is copied in 16-byte words");
static_assert(sizeof(RepHeader) % 16 == 0 && offsetof(RepHeader, cs) % 16 == 0, "RepHeader layout");

struct SlotRec { double tpf; uint32_t pk; uint32_t pad; };  // request in a decode slot: prefill end time, packed lengths/class/group
constexpr int STAGE_CAP = 64;                                 // finished-request records waiting for their accounting
// Accounting of finished requests, one block per warp (merged into the class records at kernel exit)
struct WarpClassStats { double sYm_out, sYs_out, sum_tpot; unsigned long long tok_in, tok_out; uint32_t done_mixed, done_solo; };
struct ADraw { double E; uint32_t pk; uint32_t pad; };     // one arrival draw: unit exponential (divided by the rate already when there is one block) and packed lengths
struct QEntry { double t; uint32_t pk; uint32_t cls; };   // 16 bytes: prefill queue (t = arrival) / decode buffer (t = prefill end)

struct ClassPar { double theta; uint32_t P, D, prio, pad; };
struct BlockPar { uint32_t M, pad; double xstar[MAXI], nx[MAXI], nq[MAXI], ps[MAXI], rate[MAXI], ws[MAXI], wm[MAXI]; };

// Shapes and arrays of the one-thread-per-replication family (qsim_lane.cuh); arrays are [R][...]
struct LaneSrv;
struct LanePar {
    uint32_t on;                 // this handle runs that family
    uint32_t nbk;                // calendar buckets (power of two); every pending iteration end lies less than nbk buckets ahead
    uint32_t tlev, toff[6], tsize;   // eligibility trees: internal levels, offset of every level (0 = leaves) and entries per tree
    uint32_t b8, slev, soff[5], ssize;   // slot trees: leaves per GPU, internal levels, offsets of levels 1.. and nodes per GPU
    double inv_w;                // buckets per second
    uint32_t cs_stride, smem_bytes;  // shared memory per lane for the class records (32-bit words) and per block of 1 << lsh lanes (bytes)
    LaneSrv *srv;                // [N] GPU records
    double *tarr;                // [N] arrival time of the request in prefill
    uint16_t *cal_head;          // [nbk] first GPU of every bucket
    uint32_t *cal_bm;            // [nbk/32] non-empty buckets
    uint32_t *tree;              // [3][tsize] solo decode, mixed decode, prefill
    uint32_t *sfin;              // [N][b8] finish iteration per slot (NONE32 = free)
    unsigned long long *snode;   // [N][ssize] minimum of finish << 16 | slot per group of eight
    SlotRec *srec;               // [N][B] request in each slot
    uint16_t *sfree;             // [N][B] entries at and above the GPU's decode count are its free slots
    uint32_t *pql;               // [I][qw] live bits of the prefill-queue positions
    uint32_t qw, lsh;            // words per class in pql (a multiple of four); a warp runs 1 << lsh replications in its first lanes
};

struct Params {
    uint32_t I, N, Npad, R, B, C, nblk, gate, router, placement, length_mode, qcap, hist, advance, any_theta, slots_smem;
    unsigned long long seed, rep_offset, horizon_iters, event_budget;
    double block_len;
    double coef[6];
    ClassPar cls[MAXI];
    const BlockPar *blocks;      // [nblk]
    const uint32_t *lengths;     // [I][2][LMAX] or null
    const double *inject_t;      // injected arrivals (trace replay): times [n_inject], ascending
    const uint32_t *inject_job;  // [n_inject][3] = class, P, D
    uint32_t n_inject, force_dispatch;   // force_dispatch: the policy parameters changed since the last launch
    uint32_t nchunk, launch_tag;         // nchunk > 1: the horizon of this launch is run in that many chunks per replication (see qsim_run_kernel)
    double T_abs;                // advance == 2: absolute end time of this run
    // workspace sections (all arrays are [R][...])
    RepHeader *hdr;
    char *srv;                   // per replication: server structure-of-arrays image, srv_bytes each
    uint32_t *slot_fin;          // [R][N][B]
    SlotRec *slot_rec;           // [R][N][B]
    QEntry *pq;                  // [R][I][qcap]
    QEntry *dq;                  // [R][2][qcap]
    uint32_t *hist_mem;          // [R][I][2][NBIN] or null
    uint32_t *not_done;          // [0] replications that stopped on the event budget, [1] next (chunk, replication) unit to hand out,
                                 // [2] set when a block gave up waiting for the chunk before its own
    uint32_t srv_bytes;
    uint32_t tarr_global;        // pf_tarr lives in tarr_g instead of shared memory
    double *tarr_g;              // [R][N]
    uint32_t *pfjob_g;           // [R][N] packed request in prefill, with tarr_g
    LanePar lane;
};

// ---------------------------------------------------------------------------------------------
// random numbers and elementary functions
// ---------------------------------------------------------------------------------------------

// Philox4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0,k1).
__device__ __forceinline__ void philox(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                       uint32_t &o0, uint32_t &o1, uint32_t &o2, uint32_t &o3)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    o0 = c0; o1 = c1; o2 = c2; o3 = c3;
}

__device__ __forceinline__ void draw(const Params &p, uint32_t rep, uint32_t stream, unsigned long long index,
                                     uint32_t &w0, uint32_t &w1, uint32_t &w2, uint32_t &w3)
{
    const unsigned long long grep = p.rep_offset + rep;
    philox((uint32_t)index, (uint32_t)(index >> 32), stream, (uint32_t)grep, (uint32_t)p.seed,
           (uint32_t)(p.seed >> 32), w0, w1, w2, w3);
}

// uniform on (0,1]: (top 53 bits of w0:w1, plus one) / 2^53
__device__ __forceinline__ double u53(uint32_t w0, uint32_t w1)
{
    const unsigned long long h = ((unsigned long long)w0 << 21) | (unsigned long long)(w1 >> 11);
    return __dmul_rn((double)(h + 1ull), 1.1102230246251565e-16);   // 2^-53
}

// ln x for x in (0,1] as a fixed chain of rounded operations: x = m 2^e, m in [sqrt(1/2), sqrt(2)),
// s = (m-1)/(m+1), ln m = 2 s sum_{k=0..12} s^(2k)/(2k+1), result = e ln2 + ln m.
__device__ __forceinline__ double qlog(double x)
{
    const long long bits = __double_as_longlong(x);
    int e = (int)((bits >> 52) & 0x7ff) - 1023;
    double m = __longlong_as_double((bits & 0x000fffffffffffffLL) | 0x3ff0000000000000LL);
    if (m > 1.4142135623730951) {
        m = __dmul_rn(m, 0.5);
        e += 1;
    }
    const double s = __ddiv_rn(__dsub_rn(m, 1.0), __dadd_rn(m, 1.0));
    const double z = __dmul_rn(s, s);
    // series coefficients 1/(2k+1): the correctly rounded quotients, formed once at compile time
    constexpr double inv_odd[13] = { 1.0 / 1.0, 1.0 / 3.0, 1.0 / 5.0, 1.0 / 7.0, 1.0 / 9.0, 1.0 / 11.0, 1.0 / 13.0, 1.0 / 15.0,
                                     1.0 / 17.0, 1.0 / 19.0, 1.0 / 21.0, 1.0 / 23.0, 1.0 / 25.0 };
    double acc = inv_odd[12];
#pragma unroll
    for (int k = 11; k >= 0; --k)
        acc = __dadd_rn(__dmul_rn(acc, z), inv_odd[k]);
    const double logm = __dmul_rn(__dmul_rn(2.0, s), acc);
    return __dadd_rn(__dmul_rn((double)e, 0.6931471805599453), logm);
}

// iteration time of a batch with pf prefill tokens, d decodes, K resident KV tokens (Eq. (1)-(3))
__device__ __forceinline__ double iter_time(const Params &p, uint32_t pf, uint32_t d, uint32_t K, bool kappa = true)
{
    double t;
    if (pf > 0) {
        t = __dadd_rn(p.coef[0], __dmul_rn(p.coef[1], (double)pf));
        t = __dadd_rn(t, __dmul_rn(p.coef[2], (double)d));
    } else {
        t = __dadd_rn(p.coef[3], __dmul_rn(p.coef[4], (double)d));
    }
    if (kappa && p.coef[5] != 0.0)
        t = __dadd_rn(t, __dmul_rn(p.coef[5], (double)K));
    return t;
}

__device__ __forceinline__ uint32_t hist_bin(double x)
{
    long long b = (long long)((unsigned long long)__double_as_longlong(x) >> 47) - ((long long)(1023 - 20) << 5);
    b = b < 0 ? 0 : (b > NBIN - 1 ? NBIN - 1 : b);
    return (uint32_t)b;
}

__device__ __forceinline__ uint32_t pack_job(uint32_t P, uint32_t D, uint32_t cls, uint32_t flag)
{
    return (P - 1u) | ((D - 1u) << 13) | (cls << 26) | (flag << 31);
}
__device__ __forceinline__ uint32_t job_P(uint32_t pk) { return (pk & 0x1fffu) + 1u; }
__device__ __forceinline__ uint32_t job_D(uint32_t pk) { return ((pk >> 13) & 0x1fffu) + 1u; }
__device__ __forceinline__ uint32_t job_cls(uint32_t pk) { return (pk >> 26) & 7u; }
__device__ __forceinline__ uint32_t job_flag(uint32_t pk) { return pk >> 31; }

__device__ __forceinline__ double dinf() { return __longlong_as_double(0x7ff0000000000000LL); }

__device__ __forceinline__ void area_touch(Area &a, uint32_t count, double t)
{
    a.area = __dadd_rn(a.area, __dmul_rn((double)count, __dsub_rn(t, a.t_last)));
    a.t_last = t;
}

// Abandonment clock of one (class, queue): integrated hazard acc against the exponential level lvl
// (random time change, Eq. (8)-(9)); called by the owning class lane before the count changes.
__device__ __forceinline__ void ab_change(AbClock &c, double theta, uint32_t Q_old, uint32_t Q_new, double t)
{
    if (!(theta > 0.0)) return;
    c.acc = __dadd_rn(c.acc, __dmul_rn(__dmul_rn(theta, (double)Q_old), __dsub_rn(t, c.t_last)));
    c.t_last = t;
    if (Q_new > 0) {
        double rem = __dsub_rn(c.lvl, c.acc);
        if (rem < 0.0) rem = 0.0;
        c.t_ab = __dadd_rn(t, __ddiv_rn(rem, __dmul_rn(theta, (double)Q_new)));
    } else {
        c.t_ab = dinf();
    }
}

// 16-byte asynchronous copy global -> shared (L2 only), and the wait for this thread's copies
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }
// Copies are committed one group per copy, so a thread can wait for an older copy of its own and leave the
// N groups it committed after it in flight.
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N_>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N_) : "memory"); }

// Coarse index of a threshold table: entry b = #{j < LMAX-1 : thr[j] < b 2^24}, b = 0..256 (built by the host when the
// tables are uploaded and stored behind them).  A word w with top byte b has its count between entries b and b+1.
constexpr int LIDX = 260;       // 257 entries, padded

// 1 + #{j < LMAX-1 : thr[j] <= w} by binary search inside the bucket of w's top byte
__device__ __forceinline__ uint32_t table_lookup(const uint32_t *thr, const uint16_t *idx, uint32_t w)
{
    const uint32_t b = w >> 24;
    uint32_t lo = __ldg(idx + b), hi = __ldg(idx + b + 1);          // the count lies in [lo, hi]
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (__ldg(thr + mid) <= w) lo = mid + 1; else hi = mid;
    }
    return 1u + lo;
}

// Arrival draw `index` of class i: one Philox block gives the unit exponential and both lengths.
// (Arguments by value: a reference to the kernel parameters would force a local copy of them.)
__device__ __noinline__ ADraw make_draw(unsigned long long seed, unsigned long long global_rep, uint32_t i, uint32_t I,
                                        unsigned long long index, const uint32_t *tables, uint32_t P, uint32_t D, double Lam)
{
    uint32_t w0, w1, w2, w3;
    philox((uint32_t)index, (uint32_t)(index >> 32), (STREAM_ARRIVAL << 8) | i, (uint32_t)global_rep, (uint32_t)seed,
           (uint32_t)(seed >> 32), w0, w1, w2, w3);
    ADraw d;
    d.E = -qlog(u53(w0, w1));
    if (Lam > 0.0) d.E = __ddiv_rn(d.E, Lam);      // one rate for the whole run: the interarrival time itself is stored
    if (tables) {
        const uint16_t *idx = reinterpret_cast<const uint16_t *>(tables + (size_t)I * 2 * LMAX);     // behind the tables
        P = table_lookup(tables + ((size_t)i * 2 + 0) * LMAX, idx + ((size_t)i * 2 + 0) * LIDX, w2);
        D = table_lookup(tables + ((size_t)i * 2 + 1) * LMAX, idx + ((size_t)i * 2 + 1) * LIDX, w3);
    }
    d.pk = pack_job(P, D, i, 0);
    d.pad = 0;
    return d;
}

// ---------------------------------------------------------------------------------------------
// the per-warp simulator
// ---------------------------------------------------------------------------------------------

template <int SPL, uint32_t F>
struct Sim {
    __device__ __forceinline__ bool f_abandon() const { return (F & F_GENERIC) ? p.any_theta != 0 : (F & F_ABANDON) != 0; }
    __device__ __forceinline__ bool f_sli() const { return (F & F_GENERIC) ? (p.router == 1 || p.router == 2) : (F & F_SLI) != 0; }
    __device__ __forceinline__ bool f_slig() const { return (F & F_GENERIC) ? p.router == 2 : false; }
    __device__ __forceinline__ bool f_kappa() const { return (F & F_GENERIC) ? p.coef[5] != 0.0 : (F & F_KAPPA) != 0; }
    __device__ __forceinline__ bool f_hist() const { return (F & F_GENERIC) ? hist != nullptr : (F & F_HIST) != 0; }
    __device__ __forceinline__ bool f_blocks() const { return (F & F_GENERIC) ? p.nblk > 1 : (F & F_BLOCKS) != 0; }
    __device__ __forceinline__ bool f_random() const { return (F & F_GENERIC) ? p.placement == 0 : (F & F_RANDOM) != 0; }
    __device__ __forceinline__ bool f_occ() const { return (F & F_GENERIC) ? p.gate == 0 : (F & F_OCC) != 0; }
    // finish stamps and slot occupancy of every simulated GPU live in shared memory (small N*B only)
    __device__ __forceinline__ bool f_slots() const { return (F & F_GENERIC) ? p.slots_smem != 0 : (F & F_SLOTS) != 0; }
    __device__ __forceinline__ uint32_t n_rows() const { return SPL > 0 ? (uint32_t)SPL : (p.Npad >> 5); }

    const Params &p;
    const int lane;
    const uint32_t rep;
    int warp, nwarps;            // position in the block (F_MW); 0 / 1 otherwise
    MwCmd *cmd;
    MwRes *res;
    WarpClassStats *wcs;         // [nwarps][MAXI]
    // shared memory (lane-owned entries)
    double *tnext, *pf_tarr;               // pf_tarr: arrival time of the request in prefill (shared memory, or global memory on large clusters)
    uint32_t *it, *nfin, *pfjob, *K, *Kpend;
    uint16_t *pfrem;             // prompt tokens still to prefill (0 = no request in prefill; lengths are at most 8192)
    uint16_t *ndec, *nact, *pfcur;
    uint16_t *sfin16;            // [Npad][B]  low 16 bits of each slot's finish iteration (f_slots)
    uint32_t *socc;              // [Npad][ceil(B/32)]  slot occupancy bits; bits past B are set for good
    uint32_t *touch;
    double *gate_xi, *gate_dq;
    uint32_t *gate_ok;
    ClassState *cs;
    // global memory of this replication
    uint32_t *s_fin;
    SlotRec *s_rec;
    // shared-memory staging: records of finished requests (copied asynchronously) and queue-head copies
    SlotRec *st_rec;
    double *st_te;
    QEntry *pqh;
    uint32_t n_pend;
    uint32_t rec_after;          // per lane: record copies committed since this lane's last queue-head copy
    QEntry *pq, *dq;
    uint32_t *hist;
    // replicated scalars
    double t, T_end, T_blk_next, T_reset, tau_min;
    uint32_t blk, M, dq_head0, dq_head1, dq_n0, dq_n1, n_touch, err;
    uint32_t n_idle_pf;          // mixed GPUs whose prefill slot is idle (and that may take a prefill)
    uint32_t idle_hint;          // when n_idle_pf == 1: that GPU if known, else NONE32
    uint32_t need_start;         // per lane: rows of own GPUs touched by the current event
    unsigned long long place_ord, events, rounds, sel_ord0, sel_ord1;
    bool drain_dirty, gate_dirty, touch_all;
    bool force_nonlocal;         // treat the next event, whatever it is, as non-local (it must end with a dispatch)
    // per-lane partial sums
    unsigned long long it_mixed, it_solo;
    double busy_mixed, busy_solo;
    // pre-generated arrival draws of this lane's class (ring in shared memory) and a pending scheduling request
    ADraw *aring;
    uint32_t ring_n, ring_pos;
    bool sched_pending;
    double t0_pending;
    // block parameters of the current block (lane i holds class i)
    double b_xstar, b_nx, b_nq, b_ps;

    __device__ Sim(const Params &p_, int lane_, uint32_t rep_) : p(p_), lane(lane_), rep(rep_), warp(0), nwarps(1) {}
    __device__ __forceinline__ void block_sync() const { if (F & F_MW) __syncthreads(); else __syncwarp(); }

    __device__ __forceinline__ double block_start(uint32_t b) const { return __dmul_rn((double)b, p.block_len); }

    __device__ __forceinline__ void load_block(uint32_t b)
    {
        blk = b;
        const BlockPar &bp = p.blocks[b];
        M = bp.M;
        b_xstar = 0.0; b_nx = 0.0; b_nq = 0.0; b_ps = 0.0;
        if (lane < (int)p.I) {
            b_xstar = bp.xstar[lane]; b_nx = bp.nx[lane]; b_nq = bp.nq[lane]; b_ps = bp.ps[lane];
        }
        T_blk_next = (f_blocks() && b + 1 < p.nblk) ? block_start(b + 1) : dinf();
    }

    // --- arrivals ------------------------------------------------------------------------------
    // Arrival draws do not depend on the simulation: draw k of class i is one Philox block that gives a unit
    // exponential E_k (words 0,1) and the two lengths (words 2,3).  The warp produces 32 consecutive draws
    // of a class at a time, one per lane, into a ring in shared memory; the class lane consumes them in
    // order.  Draws left in the ring at the end of a launch are given back (adraw is rewound).

    __device__ __forceinline__ void refill(uint32_t i)
    {
        const unsigned long long base = __shfl_sync(FULL, cs[lane & 7].adraw, i);
        // with a single block the class's rate never changes and the division E / Lambda is done here, 32 at a time
        const double Lam1 = f_blocks() ? 0.0 : __dmul_rn((double)p.N, p.blocks[0].rate[i]);
        aring[i * 32 + lane] = make_draw(p.seed, p.rep_offset + rep, i, p.I, base + (unsigned long long)lane,
                                         p.length_mode == 1 ? p.lengths : nullptr, p.cls[i].P, p.cls[i].D, Lam1);
        __syncwarp();
        if (lane == (int)i) {
            cs[i].adraw = base + 32ull;
            ring_pos = 0;
            ring_n = 32;
            if (sched_pending) { sched_pending = false; schedule_from(t0_pending); }
        }
        __syncwarp();
    }

    // Class lane only: next arrival of this lane's class after t0.  A candidate at or past the end of its
    // block is discarded and drawn again from the boundary under the next block's rate (memorylessness).
    __device__ void schedule_from(double t0)
    {
        ClassState &c = cs[lane];
        if ((F & F_GENERIC) && p.n_inject > 0) {
            // trace replay: the next entry of this class in the injected list (c.ablk is the read position)
            uint32_t k = c.ablk;
            while (k < p.n_inject && p.inject_job[3 * k] != (uint32_t)lane) ++k;
            if (k < p.n_inject) {
                c.ta = p.inject_t[k]; c.nextP = p.inject_job[3 * k + 1]; c.nextD = p.inject_job[3 * k + 2];
                c.ablk = k + 1;
            } else {
                c.ta = dinf(); c.ablk = k;
            }
            return;
        }
        uint32_t b = c.ablk;
        for (;;) {
            const double Lam = __dmul_rn((double)p.N, p.blocks[b].rate[lane]);
            const bool has_next = f_blocks() && b + 1 < p.nblk;
            if (!(Lam > 0.0)) {
                if (!has_next) { c.ta = dinf(); c.ablk = b; return; }
                ++b; t0 = block_start(b);
                continue;
            }
            if (ring_n == 0) {          // out of draws: the warp refills at the top of the next round
                sched_pending = true; t0_pending = t0; c.ablk = b; c.ta = dinf();
                return;
            }
            const ADraw d = aring[lane * 32 + ring_pos];
            ring_pos++; ring_n--;
            const double cand = __dadd_rn(t0, f_blocks() ? __ddiv_rn(d.E, Lam) : d.E);
            if (has_next && cand >= block_start(b + 1)) {
                ++b; t0 = block_start(b);
                continue;
            }
            c.ta = cand; c.ablk = b; c.nextP = job_P(d.pk); c.nextD = job_D(d.pk);
            return;
        }
    }

    // Class lane only: the arrival scheduled at c.ta happens; nothing outside the class is touched.
    __device__ void arrival_local()
    {
        const uint32_t i = (uint32_t)lane;
        ClassState &c = cs[i];
        const double ta = c.ta;
        c.arrivals++;
        if (c.pq_n >= p.qcap) {
            c.overflow++;
        } else {
            if (f_abandon()) ab_change(c.abp, p.cls[i].theta, c.pq_n, c.pq_n + 1, ta);
            area_touch(c.aQp, c.pq_n, ta);
            uint32_t pos = c.pq_head + c.pq_n;
            if (pos >= p.qcap) pos -= p.qcap;
            QEntry e; e.t = ta; e.pk = pack_job(c.nextP, c.nextD, i, 0); e.cls = i;
            pq[(size_t)i * p.qcap + pos] = e;
            if (c.pq_n == 0) pqh[i] = e;        // it is the head: keep a copy on chip
            c.pq_n++;
        }
        schedule_from(ta);
    }

    // warp-wide path: an arrival while some prefill slot is idle (the gate may admit it at once)
    __device__ void on_arrival(uint32_t i)
    {
        if (lane == (int)i) arrival_local();
        gate_dirty = true;
    }

    __device__ uint32_t count_idle_pf()
    {
        // per-lane count over the lane's rows (branch-free), one warp-wide sum
        uint32_t cnt = 0;
#pragma unroll 4
        for (uint32_t k = 0; k < n_rows(); ++k)
            cnt += eligible((k << 5) + (uint32_t)lane, WANT_PREFILL) ? 1u : 0u;
        return __reduce_add_sync(FULL, cnt);
    }

    // --- abandonment ---------------------------------------------------------------------------
    // Remove entry `pos` (offset from head) of a ring of n entries, keeping order: shift the tail down.
    __device__ void ring_remove(QEntry *ring, uint32_t head, uint32_t n, uint32_t pos)
    {
        const uint32_t cap = p.qcap;
        for (uint32_t k = pos; k + 1 < n; k += 32) {
            const uint32_t j = k + (uint32_t)lane;
            QEntry e;
            const bool act = j + 1 < n;
            if (act) {
                uint32_t src = head + j + 1; if (src >= cap) src -= cap;
                e = ring[src];
            }
            __syncwarp();
            if (act) {
                uint32_t dst = head + j; if (dst >= cap) dst -= cap;
                ring[dst] = e;
            }
            __syncwarp();
        }
    }

    __device__ void on_abandon_p(uint32_t i)
    {
        const uint32_t Q = __shfl_sync(FULL, cs[lane & 7].pq_n, i);
        const uint32_t head = __shfl_sync(FULL, cs[lane & 7].pq_head, i);
        const unsigned long long m = __shfl_sync(FULL, cs[lane & 7].abp.m, i);
        uint32_t w0, w1, w2, w3;
        draw(p, rep, (STREAM_ABANDON_P << 8) | i, m, w0, w1, w2, w3);
        const uint32_t rank = __umulhi(w2, Q);       // uniformly chosen waiting job, in FCFS rank
        cp_async_wait_all();
        __syncwarp();
        ring_remove(pq + (size_t)i * p.qcap, head, Q, rank);
        if (lane == (int)i) {
            ClassState &c = cs[i];
            if (Q > 1) pqh[i] = pq[(size_t)i * p.qcap + head];     // the head may have changed
            area_touch(c.aQp, Q, t);
            c.pq_n = Q - 1;
            c.abandoned_p++;
            AbClock &a = c.abp;
            a.m = m + 1; a.acc = 0.0; a.lvl = -qlog(u53(w0, w1)); a.t_last = t;
            a.t_ab = (Q - 1 > 0) ? __dadd_rn(t, __ddiv_rn(a.lvl, __dmul_rn(p.cls[i].theta, (double)(Q - 1)))) : dinf();
        }
    }

    __device__ void on_abandon_d(uint32_t pool, uint32_t i)
    {
        const uint32_t Q = __shfl_sync(FULL, pool ? cs[lane & 7].Qd1 : cs[lane & 7].Qd0, i);
        const unsigned long long m = __shfl_sync(FULL, pool ? cs[lane & 7].abd1.m : cs[lane & 7].abd0.m, i);
        uint32_t w0, w1, w2, w3;
        draw(p, rep, ((pool ? STREAM_ABANDON_D1 : STREAM_ABANDON_D0) << 8) | i, m, w0, w1, w2, w3);
        uint32_t rank = __umulhi(w2, Q);
        QEntry *ring = dq + (size_t)pool * p.qcap;
        const uint32_t head = pool ? dq_head1 : dq_head0, n = pool ? dq_n1 : dq_n0;
        // position of the rank-th class-i entry in buffer order
        uint32_t pos = NONE32;
        for (uint32_t k = 0; k < n && pos == NONE32; k += 32) {
            const uint32_t j = k + (uint32_t)lane;
            bool mine = false;
            if (j < n) {
                uint32_t src = head + j; if (src >= p.qcap) src -= p.qcap;
                mine = ring[src].cls == i;
            }
            const uint32_t b = __ballot_sync(FULL, mine);
            const uint32_t c = (uint32_t)__popc(b);
            if (rank < c) pos = k + (uint32_t)__fns(b, 0, (int)rank + 1);
            else rank -= c;
        }
        if (pos == NONE32) { err = ERR_INTERNAL; return; }
        ring_remove(ring, head, n, pos);
        if (pool) dq_n1--; else dq_n0--;
        if (lane == (int)i) {
            ClassState &c = cs[i];
            area_touch(c.aQd, c.Qd0 + c.Qd1, t);
            if (pool) c.Qd1 = Q - 1; else c.Qd0 = Q - 1;
            c.abandoned_d++;
            AbClock &a = pool ? c.abd1 : c.abd0;
            a.m = m + 1; a.acc = 0.0; a.lvl = -qlog(u53(w0, w1)); a.t_last = t;
            a.t_ab = (Q - 1 > 0) ? __dadd_rn(t, __ddiv_rn(a.lvl, __dmul_rn(p.cls[i].theta, (double)(Q - 1)))) : dinf();
        }
    }

    // --- GPU choice ----------------------------------------------------------------------------
    __device__ __forceinline__ bool eligible(uint32_t g, int want) const
    {
        // g is always inside the padded arrays; every field is read first so that calls over rows overlap
        const uint32_t nd = ndec[g];
        const bool pf = pfrem[g] != 0;
        const bool mix = g < M;
        const uint32_t cap = (mix || pf) ? p.B - 1 : p.B;   // a mixed GPU keeps one slot for prefill
        const bool ok = want == WANT_PREFILL ? (mix && !pf && nd <= p.B - 1)
                                             : ((want == WANT_MIX) == mix && nd < cap);
        return ok && g < p.N;
    }

    // uniformly at random among the eligible GPUs (k-th in index order) or least loaded, lowest index
    // Solo-first target of a decode under least-loaded placement in one reduction: key = tier, load, index.
    __device__ __forceinline__ uint32_t choose_solo_first()
    {
        uint32_t best = NONE32;
#pragma unroll 4
        for (uint32_t k = 0; k < n_rows(); ++k) {
            const uint32_t g = (k << 5) + (uint32_t)lane;
            const uint32_t nd = ndec[g];
            const bool mix = g < M;
            const uint32_t cap = (mix || pfrem[g] != 0) ? p.B - 1 : p.B;
            const uint32_t key = (mix ? 0x40000000u : 0u) | (nd << 16) | g;
            best = min(best, (nd < cap && g < p.N) ? key : NONE32);
        }
        best = __reduce_min_sync(FULL, best);
        return best == NONE32 ? NONE32 : (best & 0xffffu);
    }

    __device__ uint32_t choose_server(int want)
    {
        const uint32_t rows = n_rows();
        if (!f_random()) {
            uint32_t best = NONE32;
#pragma unroll 4
            for (uint32_t k = 0; k < rows; ++k) {
                const uint32_t g = (k << 5) + (uint32_t)lane;
                best = min(best, eligible(g, want) ? (((uint32_t)ndec[g] << 16) | g) : NONE32);
            }
            best = __reduce_min_sync(FULL, best);
            return best == NONE32 ? NONE32 : (best & 0xffffu);
        }
        uint32_t cnt = 0;
        for (uint32_t k = 0; k < rows; ++k)
            cnt += (uint32_t)__popc(__ballot_sync(FULL, eligible((k << 5) + (uint32_t)lane, want)));
        if (cnt == 0) return NONE32;
        uint32_t idx = 0;
        if (cnt > 1) {
            uint32_t w0, w1, w2, w3;
            draw(p, rep, STREAM_PLACEMENT << 8, place_ord++, w0, w1, w2, w3);
            idx = __umulhi(w0, cnt);
        }
        for (uint32_t k = 0; k < rows; ++k) {
            const uint32_t b = __ballot_sync(FULL, eligible((k << 5) + (uint32_t)lane, want));
            const uint32_t c = (uint32_t)__popc(b);
            if (idx < c) return (k << 5) + (uint32_t)__fns(b, 0, (int)idx + 1);
            idx -= c;
        }
        err = ERR_INTERNAL;
        return NONE32;
    }

    // GPU g may have to start an iteration at the end of this event: noted in its owner's row mask
    __device__ __forceinline__ void touch_server(uint32_t g)
    {
        if (SPL > 0) { if (lane == (int)(g & 31u)) need_start |= 1u << (g >> 5); }
        else if (n_touch < TOUCH_CAP) { if (lane == 0) touch[n_touch] = g; n_touch++; }
        else touch_all = true;
    }

    // --- decode placement ------------------------------------------------------------------------
    // General SLI-aware router: position (in buffer order) of the request that gets the freed slot of the pool.
    // The class is drawn with probabilities proportional to varpi over the classes that wait in the pool; one
    // waiting class needs no draw, and with no positive weight among them the head of the buffer goes.
    __device__ uint32_t select_in_pool(uint32_t pool)
    {
        const BlockPar &bp = p.blocks[blk];
        uint32_t nonempty = 0, cls = 0;
        double Wsum = 0.0;
        for (uint32_t i = 0; i < p.I; ++i)
            if ((pool ? cs[i].Qd1 : cs[i].Qd0) > 0) { ++nonempty; cls = i; Wsum = __dadd_rn(Wsum, pool ? bp.wm[i] : bp.ws[i]); }
        if (nonempty > 1) {
            if (!(Wsum > 0.0)) return 0;
            uint32_t w0, w1, w2, w3;
            if (pool) draw(p, rep, STREAM_SELECT1 << 8, sel_ord1++, w0, w1, w2, w3);
            else      draw(p, rep, STREAM_SELECT0 << 8, sel_ord0++, w0, w1, w2, w3);
            const double x = __dmul_rn(u53(w0, w1), Wsum);
            double cum = 0.0;
            uint32_t chosen = NONE32, last = NONE32;
            for (uint32_t i = 0; i < p.I && chosen == NONE32; ++i) {
                if ((pool ? cs[i].Qd1 : cs[i].Qd0) == 0) continue;
                const double w = pool ? bp.wm[i] : bp.ws[i];
                cum = __dadd_rn(cum, w);
                if (w > 0.0) { last = i; if (cum >= x) chosen = i; }
            }
            cls = chosen != NONE32 ? chosen : last;
        }
        // oldest request of the class
        const QEntry *ring = dq + (size_t)pool * p.qcap;
        const uint32_t head = pool ? dq_head1 : dq_head0, n = pool ? dq_n1 : dq_n0;
        for (uint32_t k = 0; k < n; k += 32) {
            const uint32_t j = k + (uint32_t)lane;
            bool mine = false;
            if (j < n) {
                uint32_t src = head + j; if (src >= p.qcap) src -= p.qcap;
                mine = ring[src].cls == cls;
            }
            const uint32_t b = __ballot_sync(FULL, mine);
            if (b) return k + (uint32_t)__ffs((int)b) - 1u;
        }
        err = ERR_INTERNAL;
        return 0;
    }

    // entry pos (0 = head) of the pool's buffer goes to GPU g
    __device__ void place_decode(uint32_t pool, uint32_t g, uint32_t pos = 0)
    {
        const uint32_t head = pool ? dq_head1 : dq_head0;
        QEntry *ring = dq + (size_t)pool * p.qcap;
        uint32_t src = head + pos; if (src >= p.qcap) src -= p.qcap;
        const QEntry e = ring[src];
        if (pos == 0) {
            if (pool) dq_head1 = (head + 1 == p.qcap) ? 0 : head + 1;
            else      dq_head0 = (head + 1 == p.qcap) ? 0 : head + 1;
        } else {
            __syncwarp();
            ring_remove(ring, head, pool ? dq_n1 : dq_n0, pos);
        }
        if (pool) dq_n1--; else dq_n0--;
        place_job(pool, g, e.cls, job_P(e.pk), job_D(e.pk), e.t, true);
    }

    // A request of class i whose prefill ended at tpf starts decoding on GPU g.  from_buffer: it waited in
    // the pool's buffer; otherwise it passes through the (empty) buffer at this very instant, which
    // leaves the buffer's count, integral and abandonment clock as one touch at time t would.
    __device__ void place_job(uint32_t pool, uint32_t g, uint32_t i, uint32_t P, uint32_t D, double tpf, bool from_buffer)
    {
        const bool mixed = g < M;
        if (lane == (int)i) {
            ClassState &c = cs[i];
            const uint32_t Qd = pool ? c.Qd1 : c.Qd0;
            if (f_abandon()) ab_change(pool ? c.abd1 : c.abd0, p.cls[i].theta, Qd, from_buffer ? Qd - 1 : Qd, t);
            area_touch(c.aQd, c.Qd0 + c.Qd1, t);
            if (from_buffer) { if (pool) c.Qd1--; else c.Qd0--; }
            const double rel = __dsub_rn(t, T_reset);
            if (mixed) { c.sYm_in = __dadd_rn(c.sYm_in, rel); c.Ym++; c.placed_mixed++; }
            else       { c.sYs_in = __dadd_rn(c.sYs_in, rel); c.Ys++; c.placed_solo++; }
        }
        if (lane == (int)(g & 31u)) {
            const uint32_t sl = ndec[g];
            const bool running = tnext[g] < dinf();
            // joins the iteration that starts next: a running iteration first finishes as it+1
            const uint32_t fin = it[g] + (running ? 1u : 0u) + D;
            size_t o;
            if (f_slots()) {
                // first free slot of the GPU's occupancy words
                const uint32_t bw = (p.B + 31u) >> 5;
                uint32_t slot = 0;
                for (uint32_t w = 0; w < bw; ++w) {
                    const uint32_t word = socc[g * bw + w];
                    if (word != 0xffffffffu) {
                        const uint32_t b = (uint32_t)__ffs((int)~word) - 1u;
                        socc[g * bw + w] = word | (1u << b);
                        slot = (w << 5) + b;
                        break;
                    }
                }
                sfin16[g * p.B + slot] = (uint16_t)fin;
                o = (size_t)g * p.B + slot;
            } else {
                o = (size_t)g * p.B + sl;
                s_fin[o] = fin;
            }
            SlotRec r; r.tpf = tpf; r.pk = pack_job(P, D, i, mixed ? 1u : 0u); r.pad = 0;
            s_rec[o] = r;
            ndec[g] = (uint16_t)(sl + 1);
            nfin[g] = min(nfin[g], fin);
            if (f_kappa()) Kpend[g] += P;
        }
        touch_server(g);
    }

    // --- prefill gate ------------------------------------------------------------------------------
    __device__ uint32_t gate_class()
    {
        if ((F & F_GENERIC) && p.gate == 2) {
            // FCFS ablation: the class whose head-of-line request arrived first (heads are mirrored on chip)
            cp_async_wait_all();
            __syncwarp();
            uint32_t best = NONE32;
            double bt = 0.0;
            for (uint32_t i = 0; i < p.I; ++i) {
                if (cs[i].pq_n == 0) continue;
                const double ta = pqh[i].t;
                if (best == NONE32 || ta < bt) { best = i; bt = ta; }
            }
            __syncwarp();
            return best;
        }
        if (!f_occ()) {
            // Prioritize-and-Route: largest D_i/P_i among waiting classes = smallest static rank
            uint32_t key = NONE32;
            if (lane < (int)p.I && cs[lane].pq_n > 0) key = (p.cls[lane].prio << 8) | (uint32_t)lane;
            key = __reduce_min_sync(FULL, key);
            return key == NONE32 ? NONE32 : (key & 0xffu);
        }
        if (lane < (int)p.I) {
            const ClassState &c = cs[lane];
            gate_ok[lane] = (c.pq_n > 0 && b_xstar > 0.0) ? 1u : 0u;
            gate_xi[lane] = __ddiv_rn(__dsub_rn((double)c.X, b_nx), b_xstar);   // xi_i = (X_i - n x*_i)/x*_i
            gate_dq[lane] = __dsub_rn((double)c.pq_n, b_nq);                     // Q_p,i - n q*_p,i
        }
        __syncwarp();
        uint32_t best = NONE32;
        double bxi = 0.0, bdq = 0.0;
        for (uint32_t i = 0; i < p.I; ++i) {
            if (!gate_ok[i]) continue;
            const double xi = gate_xi[i], dqv = gate_dq[i];
            if (best == NONE32 || xi < bxi || (xi == bxi && dqv > bdq)) { best = i; bxi = xi; bdq = dqv; }
        }
        __syncwarp();
        return best;
    }

    __device__ void admit(uint32_t i, uint32_t g)
    {
        // the head of the class queue is kept in shared memory (copied there asynchronously after each pop);
        // record copies of finished requests that this lane committed later stay in flight
        if (lane == (int)i) {
            if (rec_after == 1) cp_async_wait_group<1>();
            else if (rec_after == 2) cp_async_wait_group<2>();
            else cp_async_wait_group<0>();
        }
        __syncwarp();
        const QEntry e = pqh[i];
        __syncwarp();
        if (lane == (int)i) {
            ClassState &c = cs[i];
            const uint32_t head = c.pq_head;
            if (f_abandon()) ab_change(c.abp, p.cls[i].theta, c.pq_n, c.pq_n - 1, t);
            area_touch(c.aQp, c.pq_n, t);
            c.pq_n--;
            c.pq_head = (head + 1 == p.qcap) ? 0 : head + 1;
            if (c.pq_n > 0) { cp_async16(&pqh[i], &pq[(size_t)i * p.qcap + c.pq_head]); cp_async_commit(); rec_after = 0; }
            area_touch(c.aX, c.X, t);
            c.X++;
            c.admitted++;
        }
        n_idle_pf--;
        idle_hint = NONE32;
        if (lane == (int)(g & 31u)) {
            pfjob[g] = e.pk | 0x80000000u;
            pfrem[g] = (uint16_t)job_P(e.pk);
            pf_tarr[g] = e.t;
        }
        touch_server(g);
    }

    // Called by the owner: a GPU with work that is between iterations starts one at time ts.  The batch
    // (prefill chunk, decodes) is frozen here for the whole iteration, and with it what its end will bring:
    // bit 14 of nact = some decode emits its last token, bit 15 = the prefill finishes.
    // Straight-line: every field is read first and the stores are predicated on `act`, so that the calls for
    // the rows of one lane overlap.  g is always inside the padded arrays.
    __device__ __forceinline__ void start_at(uint32_t g, double ts, bool act = true)
    {
        const unsigned long long tn = (unsigned long long)__double_as_longlong(tnext[g]);
        const uint32_t nd = ndec[g], rem = pfrem[g], nf = nfin[g], it0 = it[g];
        uint32_t Kg = 0;
        if (f_kappa()) Kg = K[g] + Kpend[g];
        const bool has_pf = rem != 0;
        const uint32_t pc = has_pf ? min(p.C, rem) : 0u;
        uint32_t fl = (nf == it0 + 1u) ? 0x4000u : 0u;
        if (pc > 0 && pc == rem) fl |= 0x8000u;
        const double tau = iter_time(p, pc, nd, Kg, f_kappa());
        if (act && tn >= 0x7ff0000000000000ull && (nd > 0 || has_pf)) {
            if (f_kappa()) { K[g] = Kg; Kpend[g] = 0; }
            pfcur[g] = (uint16_t)pc;
            nact[g] = (uint16_t)(nd | fl);
            tnext[g] = __dadd_rn(ts, tau);
        }
    }
    __device__ __forceinline__ void start_if_needed(uint32_t g) { start_at(g, t); }

    __device__ void dispatch()
    {
        __syncwarp();   // queue entries and GPU state written by the event handler are visible to every lane
        // decode routing: buffered jobs first (FCFS), solo GPUs before mixed ones
        if (drain_dirty && (dq_n0 | dq_n1)) {
            if (!f_sli()) {
                while (dq_n0 > 0) {
                    uint32_t g;
                    if (!f_random()) {
                        g = choose_solo_first();
                    } else {
                        g = choose_server(WANT_SOLO);
                        if (g == NONE32) g = choose_server(WANT_MIX);
                    }
                    if (g == NONE32) break;
                    place_decode(0, g);
                    __syncwarp();
                }
            } else {
                while (dq_n0 > 0) {
                    const uint32_t g = choose_server(WANT_SOLO);
                    if (g == NONE32) break;
                    place_decode(0, g, f_slig() ? select_in_pool(0) : 0u);
                    __syncwarp();
                }
                while (dq_n1 > 0) {
                    const uint32_t g = choose_server(WANT_MIX);
                    if (g == NONE32) break;
                    place_decode(1, g, f_slig() ? select_in_pool(1) : 0u);
                    __syncwarp();
                }
            }
        }
        drain_dirty = false;
        // prefill gate on mixed GPUs whose prefill slot is idle
        if (gate_dirty) {
            while (n_idle_pf > 0) {
                if (!__any_sync(FULL, lane < (int)p.I && cs[lane & 7].pq_n > 0)) break;      // nobody waits
                const uint32_t i = gate_class();
                if (i == NONE32) break;
                // a single idle slot whose GPU is known needs no search (and draws nothing: one candidate)
                const uint32_t g = (n_idle_pf == 1 && idle_hint != NONE32) ? idle_hint : choose_server(WANT_PREFILL);
                if (g == NONE32) break;
                admit(i, g);
                __syncwarp();
            }
        }
        gate_dirty = false;
        // start the next iteration on every GPU that was touched and is between iterations
        __syncwarp();
        if (SPL > 0) {
            // every owner starts its touched GPUs; different lanes work in parallel
#pragma unroll
            for (uint32_t k = 0; k < (uint32_t)(SPL > 0 ? SPL : 1); ++k)
                start_at((k << 5) + (uint32_t)lane, t, ((need_start >> k) & 1u) != 0);
            need_start = 0;
        } else if (touch_all) {
            for (uint32_t k = 0; k < n_rows(); ++k) {
                const uint32_t g = (k << 5) + (uint32_t)lane;
                if (g < p.N) start_if_needed(g);
            }
        } else {
            // one lane per touched GPU (a GPU noted twice is started by two lanes with the same result)
            for (uint32_t k = (uint32_t)lane; k < n_touch; k += 32u) start_if_needed(touch[k]);
        }
        n_touch = 0;
        touch_all = false;
    }

    // Some decode on GPU g emitted its last token in the iteration that ended at te (its it-th): the whole
    // warp scans the GPU's slot list from the tail, accounts every finished request and closes the gaps.
    // Accounting of one finished request (uniform arguments; the class lane does the work).
    __device__ __forceinline__ void account_done(uint32_t pk, double tpf, double te)
    {
        const uint32_t i = job_cls(pk), P = job_P(pk), D = job_D(pk);
        if (lane == (int)i) {
            WarpClassStats &c = wcs[warp * MAXI + (int)i];
            const double rel = __dsub_rn(te, T_reset);
            if (job_flag(pk)) { c.sYm_out = __dadd_rn(c.sYm_out, rel); c.done_mixed++; }
            else              { c.sYs_out = __dadd_rn(c.sYs_out, rel); c.done_solo++; }
            c.tok_in += P;       // bundled charging credits the request here, Eq. (21)-(22)
            c.tok_out += D;
            const double tpot = __ddiv_rn(__dsub_rn(te, tpf), (double)D);
            c.sum_tpot = __dadd_rn(c.sum_tpot, tpot);
            if (f_hist()) atomicAdd(&hist[((size_t)i * 2 + 1) * NBIN + hist_bin(tpot)], 1u);
        }
    }

    // Accounting of the finished requests whose records were staged in shared memory.
    __device__ void flush_done()
    {
        cp_async_wait_all();
        __syncwarp();
        for (uint32_t e = 0; e < n_pend; ++e) {
            const SlotRec r = st_rec[e];
            account_done(r.pk, r.tpf, st_te[e]);
        }
        n_pend = 0;
        __syncwarp();
    }

    // retire_decodes when stamps and occupancy are in shared memory: every lane checks one slot per word of
    // occupancy; the lanes that hit fetch their request records at the same time.
    __device__ void retire_slots(uint32_t g, uint32_t itg, uint32_t nd, double te)
    {
        const int owner = (int)(g & 31u);
        const uint32_t bw = (p.B + 31u) >> 5, it16 = itg & 0xffffu;
        uint32_t newmin = NONE32, done = 0, Kdrop = 0;
        for (uint32_t w = 0; w < bw; ++w) {
            const uint32_t occ = socc[g * bw + w];
            const uint32_t j = (w << 5) + (uint32_t)lane;
            const bool live = ((occ >> lane) & 1u) != 0 && j < p.B;
            const uint32_t dist = live ? (((uint32_t)sfin16[g * p.B + j] - it16) & 0xffffu) : NONE32;
            const bool hit = live && dist == 0;
            if (live && !hit) newmin = min(newmin, dist);
            uint32_t hits = __ballot_sync(FULL, hit);
            if (hits) {
                if (lane == owner) socc[g * bw + w] = occ & ~hits;
                done += (uint32_t)__popc(hits);
                if (!f_kappa()) {
                    // the records only feed statistics: copy them on chip asynchronously, account later
                    if (n_pend + 32u > (uint32_t)STAGE_CAP) flush_done();
                    if (hit) {
                        const uint32_t pos = n_pend + (uint32_t)__popc(hits & ((1u << lane) - 1u));
                        cp_async16(&st_rec[pos], &s_rec[(size_t)g * p.B + j]);
                        cp_async_commit();
                        rec_after++;
                        st_te[pos] = te;
                    }
                    n_pend += (uint32_t)__popc(hits);
                } else {
                    SlotRec r; r.tpf = 0.0; r.pk = 0;
                    if (hit) r = s_rec[(size_t)g * p.B + j];
                    while (hits) {
                        const int hl = __ffs((int)hits) - 1;
                        hits &= hits - 1;
                        const uint32_t pkh = __shfl_sync(FULL, r.pk, hl);
                        const double tpfh = __shfl_sync(FULL, r.tpf, hl);
                        account_done(pkh, tpfh, te);
                        Kdrop += job_P(pkh) + job_D(pkh);
                    }
                }
            }
        }
        newmin = __reduce_min_sync(FULL, newmin);
        if (lane == owner) {
            ndec[g] = (uint16_t)(nd - done);
            nfin[g] = newmin == NONE32 ? NONE32 : itg + newmin;
            if (f_kappa()) K[g] -= Kdrop;
        }
        __syncwarp();
    }

    __device__ void retire_decodes(uint32_t g, uint32_t itg, uint32_t nd, double te)
    {
        if (f_slots()) { retire_slots(g, itg, nd, te); return; }
        const int owner = (int)(g & 31u);
        uint32_t n = nd, newmin = NONE32, Kdrop = 0;
        const size_t base = (size_t)g * p.B;
        for (int k = (int)((nd - 1) >> 5); k >= 0; --k) {
            const uint32_t j = ((uint32_t)k << 5) + (uint32_t)lane;
            const uint32_t f = j < nd ? s_fin[base + j] : NONE32;
            const bool hit = f == itg;
            if (!hit) newmin = min(newmin, f);
            uint32_t hits = __ballot_sync(FULL, hit);
            while (hits) {
                const int hl = 31 - __clz(hits);
                hits &= ~(1u << hl);
                const uint32_t h = ((uint32_t)k << 5) + (uint32_t)hl;
                const SlotRec rh = s_rec[base + h];
                account_done(rh.pk, rh.tpf, te);
                Kdrop += job_P(rh.pk) + job_D(rh.pk);
                const uint32_t last = n - 1;
                __syncwarp();
                if (lane == 0 && h != last) {
                    s_fin[base + h] = s_fin[base + last];
                    s_rec[base + h] = s_rec[base + last];
                }
                n = last;
            }
        }
        newmin = __reduce_min_sync(FULL, newmin);
        if (lane == owner) {
            ndec[g] = (uint16_t)n;
            nfin[g] = newmin;
            if (f_kappa()) K[g] -= Kdrop;
        }
        __syncwarp();
    }

    // --- end of an iteration on GPU g (warp-wide path: the end is not local) ----------------------
    __device__ void on_server(uint32_t g)
    {
        const int owner = (int)(g & 31u);
        uint32_t flags = 0, itg = 0, nd = 0;
        bool recount_idle = false;
        if (SPL > 0) {
            // the round's passes have ended the iteration and retired its finished decodes; the frozen batch
            // flags say what the end brought
            const uint32_t na = nact[g];
            flags = ((na >> 14) & 1u) | (((na >> 15) & 1u) << 1);
        } else {
            if (lane == owner) {
                itg = it[g] + 1;
                it[g] = itg;
                const uint32_t na = nact[g] & 0x3fffu, pc = pfcur[g], Kg = f_kappa() ? K[g] : 0u;
                const double tau = iter_time(p, pc, na, Kg, f_kappa());     // duration of the iteration that ends (the chain of its start)
                if (pc > 0) { it_mixed++; busy_mixed = __dadd_rn(busy_mixed, tau); }
                else        { it_solo++;  busy_solo = __dadd_rn(busy_solo, tau); }
                if (f_kappa()) K[g] = Kg + na;
                tnext[g] = dinf();
                nd = ndec[g];
                if (nfin[g] == itg) flags |= 1u;
                if (pc > 0) {
                    const uint32_t rem = pfrem[g] - pc;
                    pfrem[g] = (uint16_t)rem;
                    if (rem == 0) flags |= 2u;
                }
                pfcur[g] = 0;
            }
            flags = __shfl_sync(FULL, flags, owner);
            if (flags & 1u) {
                itg = __shfl_sync(FULL, itg, owner);
                nd = __shfl_sync(FULL, nd, owner);
                retire_decodes(g, itg, nd, t);
            }
        }
        if (flags & 1u) {
            drain_dirty = true;
            gate_dirty = true;   // a promoted GPU at the cap may now take a prefill
            if (SPL > 0) {
                recount_idle = true;
            } else if (!(flags & 2u) && g < M && pfrem[g] == 0 && nd > p.B - 1 && ndec[g] <= p.B - 1) {
                // Only g changed: its idle prefill slot counts again once its decodes fit under the mixed cap (a prefill
                // that finishes in this event is counted below, with the decode count after the retirement).
                n_idle_pf++;
                idle_hint = (n_idle_pf == 1) ? g : NONE32;
            }
        }
        if (flags & 2u) {
            // prefill finished: account, then hand the request to the decode stage
            const uint32_t pk = pfjob[g];
            const double tarr = pf_tarr[g];
            const uint32_t i = job_cls(pk), P = job_P(pk), D = job_D(pk);
            uint32_t pool = 0;
            if (f_sli()) {
                // SLI-aware router: one uniform per finished prefill decides the pool
                const unsigned long long ord = __shfl_sync(FULL, cs[lane & 7].sli_ord, i);
                const double ps = __shfl_sync(FULL, b_ps, i);
                uint32_t w0, w1, w2, w3;
                draw(p, rep, (STREAM_SLI << 8) | i, ord, w0, w1, w2, w3);
                pool = (u53(w0, w1) <= ps) ? 0u : 1u;
            }
            if (lane == (int)i) {
                ClassState &c = cs[i];
                area_touch(c.aX, c.X, t);
                c.X--;
                c.prefill_done++;
                c.tok_in_pf += P;                  // separate charging credits the prompt here, Eq. (23)
                const double ttft = __dsub_rn(t, tarr);
                c.sum_ttft = __dadd_rn(c.sum_ttft, ttft);
                if (f_hist()) atomicAdd(&hist[((size_t)i * 2 + 0) * NBIN + hist_bin(ttft)], 1u);
                if (f_sli()) c.sli_ord++;
            }
            __syncwarp();   // every lane has read the finished job before its owner clears it
            if (lane == owner) pfjob[g] = 0;
            __syncwarp();
            // No router (immediate same-slot decoding, an ablation of the paper's EC): the request goes on decoding on
            // g, in the slot it holds; it passes through the empty buffer at this instant.
            const bool immediate = (F & F_GENERIC) && p.router == 3;
            if (immediate) {
                place_job(0, g, i, P, D, t, false);
                __syncwarp();
            }
            // the prefill slot of g is idle again
            if (!recount_idle && g < M && ndec[g] <= p.B - 1) {
                n_idle_pf++;
                idle_hint = (n_idle_pf == 1) ? g : NONE32;
            }
            // Decode stage.  With an empty buffer the request is its head at once: place it if a slot is free.
            const uint32_t n = pool ? dq_n1 : dq_n0;
            bool placed = immediate;
            if (!immediate && n == 0) {
                uint32_t h;
                if (f_sli()) {
                    h = choose_server(pool == 0 ? WANT_SOLO : WANT_MIX);
                } else if (!f_random()) {
                    h = choose_solo_first();
                } else {
                    h = choose_server(WANT_SOLO);
                    if (h == NONE32) h = choose_server(WANT_MIX);
                }
                if (h != NONE32) { place_job(pool, h, i, P, D, t, false); placed = true; }
            }
            if (!placed) {
                const bool full = n >= p.qcap;
                if (lane == (int)i) {
                    ClassState &c = cs[i];
                    if (full) {
                        c.overflow_d++;
                    } else {
                        const uint32_t Qd = pool ? c.Qd1 : c.Qd0;
                        if (f_abandon()) ab_change(pool ? c.abd1 : c.abd0, p.cls[i].theta, Qd, Qd + 1, t);
                        area_touch(c.aQd, c.Qd0 + c.Qd1, t);
                        if (pool) c.Qd1++; else c.Qd0++;
                    }
                }
                if (!full) {
                    uint32_t pos = (pool ? dq_head1 : dq_head0) + n;
                    if (pos >= p.qcap) pos -= p.qcap;
                    if (lane == 0) {
                        QEntry e; e.t = t; e.pk = pack_job(P, D, i, 0); e.cls = i;
                        dq[(size_t)pool * p.qcap + pos] = e;
                    }
                    if (pool) dq_n1++; else dq_n0++;
                }
                drain_dirty = true;
            }
            gate_dirty = true;
        }
        if (recount_idle) { __syncwarp(); n_idle_pf = count_idle_pf(); idle_hint = NONE32; }
        touch_server(g);
    }

    // --- local end of an iteration (owner lane only) ----------------------------------------------------
    // The iteration of GPU g ends at te and nothing outside g depends on it.  Returns true when a decode
    // finished: the GPU then waits for retire_decodes before it starts its next iteration.
    // evt: the end is the round's non-local event; the GPU is then not restarted here (the event's handler and
    // the dispatch that follows may change its batch first).
    __device__ __forceinline__ bool local_end(uint32_t g, double te, bool act = true, bool evt = false)
    {
        // straight-line: all fields are read first and the stores are predicated on `act` (see start_at)
        const uint32_t it0 = it[g], na_raw = nact[g], pc = pfcur[g], nd = ndec[g], pr = pfrem[g], nf = nfin[g];
        uint32_t K0 = 0, Kp = 0;
        if (f_kappa()) { K0 = K[g]; Kp = Kpend[g]; }
        const double tau = iter_time(p, pc, na_raw & 0x3fffu, K0, f_kappa());   // duration of the iteration that ends (the chain of its start)
        const uint32_t itg = it0 + 1u;
        const uint32_t rem = pr - pc;                       // prompt tokens left after this iteration's chunk
        const bool retire = (na_raw & 0x4000u) != 0;        // a decode finished: the GPU waits for retire_decodes
        const bool has_pf = rem != 0;                       // (the end of a prefill is never local: rem > 0 while one runs)
        const bool restart = !retire && !evt && (nd != 0 || has_pf);
        // restart at te with what the GPU holds now (requests placed meanwhile join here)
        const uint32_t Kend = K0 + (na_raw & 0x3fffu);
        const uint32_t Kg = Kend + Kp;
        const uint32_t pc2 = has_pf ? min(p.C, rem) : 0u;
        uint32_t fl = (nf == itg + 1u) ? 0x4000u : 0u;
        if (pc2 > 0 && pc2 == rem) fl |= 0x8000u;
        const double tau2 = iter_time(p, pc2, nd, Kg, f_kappa());
        if (act) {
            it[g] = itg;
            if (pc > 0) { it_mixed++; busy_mixed = __dadd_rn(busy_mixed, tau); pfrem[g] = (uint16_t)rem; }
            else        { it_solo++;  busy_solo = __dadd_rn(busy_solo, tau); }
            if (f_kappa()) { K[g] = restart ? Kg : Kend; if (restart) Kpend[g] = 0; }
            pfcur[g] = restart ? (uint16_t)pc2 : (uint16_t)0;
            if (restart) nact[g] = (uint16_t)(nd | fl);
            tnext[g] = restart ? __dadd_rn(te, tau2) : dinf();
        }
        return act && retire;
    }

    // Class lanes of the master: add every warp's accounting of finished requests to the class records.
    __device__ void merge_warp_stats()
    {
        if (warp == 0 && lane < (int)p.I) {
            ClassState &c = cs[lane];
            for (int w = 0; w < nwarps; ++w) {
                const WarpClassStats &a = wcs[w * MAXI + lane];
                c.sYm_out = __dadd_rn(c.sYm_out, a.sYm_out);
                c.sYs_out = __dadd_rn(c.sYs_out, a.sYs_out);
                c.sum_tpot = __dadd_rn(c.sum_tpot, a.sum_tpot);
                c.tok_in_done += a.tok_in; c.tok_out_done += a.tok_out;
                c.done_mixed += a.done_mixed; c.done_solo += a.done_solo;
                c.Ym -= a.done_mixed; c.Ys -= a.done_solo;
            }
        }
    }

    // This warp's share (rows warp, warp + nwarps, ...) of the candidate scan; run-time row count.
    __device__ void scan_share(bool buffered, unsigned long long &bt, uint32_t &bs, unsigned long long &tmin)
    {
        const unsigned long long INF = 0x7ff0000000000000ull;
#pragma unroll 4
        for (uint32_t k = (uint32_t)warp; k < n_rows(); k += (uint32_t)nwarps) {
            // straight-line (INF is the identity of the minimum; padded GPUs never run)
            const uint32_t g = (k << 5) + (uint32_t)lane;
            const unsigned long long v = (unsigned long long)__double_as_longlong(tnext[g]);
            const uint32_t na = nact[g], nd = ndec[g];
            const bool nl = force_nonlocal || (na & 0x8000u) != 0 ||
                            ((na & 0x4000u) != 0 && (buffered || (g < M && nd > p.B - 1)));
            tmin = min(tmin, v);
            if (v < INF && nl && v < bt) { bt = v; bs = SRC_SERVER + g; }
        }
    }

    // This warp's share of the local iteration ends below the limit key, with their retirements.
    __device__ bool ends_share(unsigned long long lim_t, uint32_t lim_s, bool buffered)
    {
        bool progressed = false;
        for (uint32_t k = (uint32_t)warp; k < n_rows(); k += (uint32_t)nwarps) {
            const uint32_t g = (k << 5) + (uint32_t)lane;
            const unsigned long long v = (unsigned long long)__double_as_longlong(tnext[g]);
            bool retire = false;
            if ((v < lim_t || (v == lim_t && SRC_SERVER + g < lim_s)) && is_local(g, buffered)) {     // (the limit is finite)
                retire = local_end(g, __longlong_as_double((long long)v));
                progressed = true;
            }
            uint32_t need = __ballot_sync(FULL, retire);
            __syncwarp();   // the owners' updates of it / n_dec are visible to the whole warp
            while (need) {
                const int l = __ffs((int)need) - 1;
                need &= need - 1;
                const uint32_t gg = (k << 5) + (uint32_t)l;
                const double te = __longlong_as_double((long long)__shfl_sync(FULL, v, l));
                retire_decodes(gg, it[gg], (uint32_t)ndec[gg], te);
                if (lane == l) start_at(gg, te);
            }
        }
        return progressed;
    }

    // warp-level argmin of (time bits, source) and min of times
    __device__ __forceinline__ void warp_keys(unsigned long long bt, uint32_t bs, unsigned long long tmin,
                                              unsigned long long &tint, uint32_t &src, unsigned long long &tmin_all) const
    {
        const uint32_t hi = (uint32_t)(bt >> 32), lo = (uint32_t)bt;
        const uint32_t mhi = __reduce_min_sync(FULL, hi);
        const uint32_t mlo = __reduce_min_sync(FULL, hi == mhi ? lo : NONE32);
        src = __reduce_min_sync(FULL, (hi == mhi && lo == mlo) ? bs : NONE32);
        tint = ((unsigned long long)mhi << 32) | mlo;
        const uint32_t th = (uint32_t)(tmin >> 32);
        const uint32_t tmh = __reduce_min_sync(FULL, th);
        const uint32_t tml = __reduce_min_sync(FULL, th == tmh ? (uint32_t)tmin : NONE32);
        tmin_all = ((unsigned long long)tmh << 32) | tml;
    }

    // Helper warps (F_MW): serve the master's commands until it says stop.  Every command is bracketed by two
    // block barriers; the master executes the same two.
    __device__ void helper_loop()
    {
        const unsigned long long INF = 0x7ff0000000000000ull;
        for (;;) {
            __syncthreads();
            const uint32_t op = cmd->op;
            if (op == MW_EXIT) return;
            const bool buffered = cmd->buffered != 0;
            M = cmd->M;
            force_nonlocal = cmd->force != 0;
            if (op == MW_SCAN) {
                unsigned long long bt = INF, tmin = INF, tint, tall;
                uint32_t bs = NONE32, src;
                scan_share(buffered, bt, bs, tmin);
                warp_keys(bt, bs, tmin, tint, src, tall);
                if (lane == 0) { MwRes r; r.bt = tint; r.bs = src; r.tmin = tall; r.progressed = 0; res[warp] = r; }
            } else {
                const bool pr = ends_share(cmd->lim_t, cmd->lim_s, buffered);
                const uint32_t any = __ballot_sync(FULL, pr);
                if (lane == 0) res[warp].progressed = any != 0;
            }
            __syncthreads();
        }
    }

    // --- round loop ----------------------------------------------------------------------------------
    __device__ bool run()
    {
        const uint32_t rows = n_rows();
        const unsigned long long INF = 0x7ff0000000000000ull;
        const unsigned long long tend_bits = (unsigned long long)__double_as_longlong(T_end);
        unsigned long long budget = p.event_budget;
        for (;;) {
            __syncwarp();
            // classes that ran out of arrival draws get 32 new ones
            for (uint32_t need = __ballot_sync(FULL, sched_pending); need; need &= need - 1)
                refill((uint32_t)__ffs((int)need) - 1u);
            // next non-local event of this lane (sources scanned in id order with '<' keep the tie order);
            // an arrival is local while no prefill slot is idle: it only joins its class queue
            unsigned long long bt = INF, tmin = INF;
            uint32_t bs = NONE32;
            if (f_blocks() && lane == 0 && T_blk_next < dinf()) { bt = (unsigned long long)__double_as_longlong(T_blk_next); bs = SRC_BLOCK; }
            if (lane < (int)p.I) {
                const ClassState &c = cs[lane];
                unsigned long long v = (unsigned long long)__double_as_longlong(c.ta);
                tmin = v;
                if ((n_idle_pf > 0 || force_nonlocal) && v < bt) { bt = v; bs = SRC_ARRIVAL + lane; }
                if (f_abandon()) {
                    v = (unsigned long long)__double_as_longlong(c.abp.t_ab);
                    if (v < bt) { bt = v; bs = SRC_ABP + lane; }
                    v = (unsigned long long)__double_as_longlong(c.abd0.t_ab);
                    if (v < bt) { bt = v; bs = SRC_ABD0 + lane; }
                    v = (unsigned long long)__double_as_longlong(c.abd1.t_ab);
                    if (v < bt) { bt = v; bs = SRC_ABD1 + lane; }
                }
            }
            const bool buffered = (dq_n0 | dq_n1) != 0;
            constexpr int NC = SPL > 0 ? SPL : 1;       // per-row values kept in registers when the rows unroll
            unsigned long long vrow[NC];
            bool lrow[NC];
            unsigned long long tint, tmin_all;
            uint32_t src;
            if (F & F_MW) {
                // every warp scans its rows; the partial results meet in shared memory
                if (lane == 0) { cmd->op = MW_SCAN; cmd->buffered = buffered; cmd->M = M; cmd->force = force_nonlocal; }
                __syncthreads();
                scan_share(buffered, bt, bs, tmin);
                warp_keys(bt, bs, tmin, tint, src, tmin_all);
                if (lane == 0) { MwRes r; r.bt = tint; r.bs = src; r.tmin = tmin_all; r.progressed = 0; res[0] = r; }
                __syncthreads();
                bt = INF; bs = NONE32; tmin = INF;
                if (lane < nwarps) { bt = res[lane].bt; bs = res[lane].bs; tmin = res[lane].tmin; }
                warp_keys(bt, bs, tmin, tint, src, tmin_all);
            } else {
#pragma unroll
                for (uint32_t k = 0; k < rows; ++k) {
                    // straight-line (INF is the identity of the minimum; padded GPUs never run)
                    const uint32_t g = (k << 5) + (uint32_t)lane;
                    const unsigned long long v = (unsigned long long)__double_as_longlong(tnext[g]);
                    const uint32_t na = nact[g], nd = ndec[g];
                    const bool nl = force_nonlocal || (na & 0x8000u) != 0 ||
                                    ((na & 0x4000u) != 0 && (buffered || (g < M && nd > p.B - 1)));
                    const bool loc = v < INF && !nl;
                    if (SPL > 0) { vrow[k] = v; lrow[k] = loc; }
                    tmin = min(tmin, v);
                    if (v < INF && nl && v < bt) { bt = v; bs = SRC_SERVER + g; }
                }
                // warp argmin of (time bits, source id) over non-local events; warp min over all pending times
                warp_keys(bt, bs, tmin, tint, src, tmin_all);
            }
            if (tint > tend_bits && tmin_all > tend_bits) return true;     // nothing left up to T_end
            if (budget == 0) return false;
            --budget;
            ++rounds;
            // no iteration that starts in this round can end before T_min + tau_min
            unsigned long long wt = INF;
            if (tmin_all < INF)
                wt = (unsigned long long)__double_as_longlong(__dadd_rn(__longlong_as_double((long long)tmin_all), tau_min));
            // local ends strictly before the limit key min{(T_int, src), (W, 0), (T_end, max)}
            unsigned long long lim_t = tint;
            uint32_t lim_s = src;
            if (wt <= lim_t) { lim_t = wt; lim_s = 0; }
            if (tend_bits < lim_t) { lim_t = tend_bits; lim_s = NONE32; }
            bool progressed = false;
            if (F & F_MW) {
                if (lane == 0) { cmd->op = MW_ENDS; cmd->lim_t = lim_t; cmd->lim_s = lim_s; cmd->buffered = buffered; cmd->M = M; cmd->force = force_nonlocal; }
                __syncthreads();
            }
            if (lane < (int)p.I && n_idle_pf == 0 && !force_nonlocal) {
                // local arrivals of this lane's class, in time order, up to the limit and up to the class's own
                // next abandonment (which each arrival moves)
                ClassState &c = cs[lane];
                for (int guard = 0; guard < 64; ++guard) {
                    const unsigned long long v = (unsigned long long)__double_as_longlong(c.ta);
                    if (!(v < lim_t || (v == lim_t && SRC_ARRIVAL + (uint32_t)lane < lim_s))) break;
                    if (f_abandon() && v > (unsigned long long)__double_as_longlong(c.abp.t_ab)) break;
                    arrival_local();
                    progressed = true;
                }
            }
            // a class that ran out of draws has an unknown next arrival, possibly before T_int, and a local
            // arrival may have pulled its class's next abandonment before T_int: then T_int is not next after all
            bool redo = sched_pending;
            if (f_abandon() && lane < (int)p.I) {
                const unsigned long long v = (unsigned long long)__double_as_longlong(cs[lane].abp.t_ab);
                redo = redo || v < tint || (v == tint && SRC_ABP + (uint32_t)lane < src);
            }
            // the non-local event happens in this round if it comes before anything a new iteration could bring
            const bool any_redo = __any_sync(FULL, redo);
            const bool do_event = !any_redo && tint < wt && tint <= tend_bits;
            // with unrolled rows the event GPU's iteration ends in pass 1 and its decodes retire in pass 2
            const uint32_t ev_g = (SPL > 0 && do_event && src >= SRC_SERVER) ? src - SRC_SERVER : NONE32;
            // pass 1: every lane ends the local iterations of its own GPUs (straight-line over the rows)
            uint32_t retire_rows = 0;
            if (SPL == 0) {
                // run-time row count (and, with helpers, only this warp's rows): ends and retirements row by row
                if (ends_share(lim_t, lim_s, buffered)) progressed = true;
                if (F & F_MW) {
                    const uint32_t mine = __ballot_sync(FULL, progressed);
                    if (lane == 0) res[0].progressed = mine != 0;
                    __syncthreads();
                    if (lane < nwarps && res[lane].progressed) progressed = true;
                }
            }
            if (SPL > 0) {
#pragma unroll
                for (uint32_t k = 0; k < rows; ++k) {
                    const uint32_t g = (k << 5) + (uint32_t)lane;
                    const unsigned long long v = vrow[k];
                    const bool evt = g == ev_g;
                    const bool act = evt || (lrow[k] && (v < lim_t || (v == lim_t && SRC_SERVER + g < lim_s)));
                    if (local_end(g, __longlong_as_double((long long)v), act, evt)) retire_rows |= 1u << k;
                    progressed = progressed || act;
                }
            }
            if (SPL > 0) {
                // pass 2: decode completions found in pass 1, retired by the whole warp, GPU by GPU
                if (__ballot_sync(FULL, retire_rows != 0)) {
                    __syncwarp();   // the owners' updates of it / n_dec are visible to the whole warp
#pragma unroll
                    for (uint32_t k = 0; k < rows; ++k) {
                        uint32_t need = __ballot_sync(FULL, (retire_rows >> k) & 1u);
                        while (need) {
                            const int l = __ffs((int)need) - 1;
                            need &= need - 1;
                            const uint32_t gg = (k << 5) + (uint32_t)l;
                            const double te = __longlong_as_double((long long)__shfl_sync(FULL, vrow[k], l));
                            retire_decodes(gg, it[gg], (uint32_t)ndec[gg], te);
                        }
                    }
                    // the retired GPUs restart where their iteration ended (straight-line over the rows)
#pragma unroll
                    for (uint32_t k = 0; k < rows; ++k)
                        start_at((k << 5) + (uint32_t)lane, __longlong_as_double((long long)vrow[k]),
                                 ((retire_rows >> k) & 1u) != 0 && (k << 5) + (uint32_t)lane != ev_g);
                }
            }
            if (do_event) {
                t = __longlong_as_double((long long)tint);
                if (src >= SRC_SERVER) {
                    on_server(src - SRC_SERVER);
                } else {
                    if (f_abandon() && src >= SRC_ABD1) on_abandon_d(1, src - SRC_ABD1);
                    else if (f_abandon() && src >= SRC_ABD0) on_abandon_d(0, src - SRC_ABD0);
                    else if (f_abandon() && src >= SRC_ABP) on_abandon_p(src - SRC_ABP);
                    else if (src >= SRC_ARRIVAL) on_arrival(src - SRC_ARRIVAL);
                    else { ++events; load_block(blk + 1); drain_dirty = true; gate_dirty = true; n_idle_pf = count_idle_pf(); idle_hint = NONE32; }
                }
                if (err) return true;
                dispatch();
                force_nonlocal = false;
            } else if (!any_redo && !__any_sync(FULL, progressed)) {
                err = ERR_INTERNAL;     // a round that neither ended an iteration nor handled an event: never spin
                return true;
            }
        }
    }

    // Is the end of the running iteration of GPU g local?  Not when its prefill finishes, nor when a decode
    // finishes while requests wait in a decode buffer or while the GPU (moved into the mixed group by a block
    // switch) holds a full solo batch and could take a prefill afterwards.
    __device__ __forceinline__ bool is_local(uint32_t g, bool buffered) const
    {
        if (force_nonlocal) return false;
        const uint32_t na = nact[g];
        if (na & 0x8000u) return false;
        if ((na & 0x4000u) && (buffered || (g < M && ndec[g] > p.B - 1))) return false;
        return true;
    }
};

// shared-memory carve-up for one replication (one warp per block)
struct SmemLayout {
    uint32_t off_tnext, off_tarr, off_it, off_nfin, off_pfrem, off_pfjob, off_K, off_Kpend, off_ndec, off_nact,
        off_pfcur, off_sfin16, off_socc, srv_bytes, off_touch, off_gate, off_cs, off_ring, off_strec, off_stte, off_pqh, off_wcs, off_cmd, off_res, total;
};

// tarr_global: the arrival times and the job words of the requests in prefill (read once per finished prefill) live in
// global memory (large clusters: shared memory is what limits the resident replications there); I: classes (sizes the
// class records and the ring of arrival draws)
__host__ __device__ inline SmemLayout smem_layout(uint32_t Npad, uint32_t B, uint32_t slots_smem, uint32_t nwarps, bool kappa,
                                                  bool tarr_global, uint32_t I)
{
    SmemLayout L;
    uint32_t o = 0;
    L.off_tnext = o; o += 8 * Npad;
    L.off_tarr = o; if (!tarr_global) o += 8 * Npad;
    L.off_it = o; o += 4 * Npad;
    L.off_nfin = o; o += 4 * Npad;
    L.off_pfjob = o; if (!tarr_global) o += 4 * Npad;
    L.off_K = o; if (kappa) o += 4 * Npad;        // KV-token counts exist only when the KV slope is on
    L.off_Kpend = o; if (kappa) o += 4 * Npad;
    L.off_ndec = o; o += 2 * Npad;
    L.off_nact = o; o += 2 * Npad;
    L.off_pfcur = o; o += 2 * Npad;
    L.off_pfrem = o; o += 2 * Npad;
    o = (o + 15u) & ~15u;
    L.off_sfin16 = o; if (slots_smem) o += 2 * Npad * B;
    o = (o + 15u) & ~15u;
    L.off_socc = o; if (slots_smem) o += 4 * Npad * ((B + 31u) >> 5);
    o = (o + 15u) & ~15u;
    L.srv_bytes = o;
    L.off_touch = o; o += 4 * TOUCH_CAP;
    o = (o + 7u) & ~7u;
    L.off_gate = o; o += (8 + 8 + 4) * MAXI;
    o = (o + 15u) & ~15u;
    L.off_cs = o; o += (uint32_t)sizeof(ClassState) * I;
    o = (o + 15u) & ~15u;
    L.off_ring = o; o += (uint32_t)sizeof(ADraw) * 32 * I;
    L.off_strec = o; o += (uint32_t)sizeof(SlotRec) * STAGE_CAP;
    L.off_stte = o; o += 8 * STAGE_CAP;
    L.off_pqh = o; o += (uint32_t)sizeof(QEntry) * MAXI;
    L.off_wcs = o; o += (uint32_t)sizeof(WarpClassStats) * MAXI * nwarps;
    o = (o + 15u) & ~15u;
    L.off_cmd = o; if (nwarps > 1) o += (uint32_t)sizeof(MwCmd);        // master and helpers only
    o = (o + 15u) & ~15u;
    L.off_res = o; if (nwarps > 1) o += (uint32_t)sizeof(MwRes) * MW_MAX;
    L.total = (o + 15u) & ~15u;
    return L;
}

template <int SPL, uint32_t F>
__device__ __forceinline__ void bind_pointers(Sim<SPL, F> &s, char *sm, const SmemLayout &L)
{
    s.tnext = reinterpret_cast<double *>(sm + L.off_tnext);
    s.pf_tarr = s.p.tarr_global ? s.p.tarr_g + (size_t)s.rep * s.p.N : reinterpret_cast<double *>(sm + L.off_tarr);
    s.it = reinterpret_cast<uint32_t *>(sm + L.off_it);
    s.nfin = reinterpret_cast<uint32_t *>(sm + L.off_nfin);
    s.pfrem = reinterpret_cast<uint16_t *>(sm + L.off_pfrem);
    s.pfjob = s.p.tarr_global ? s.p.pfjob_g + (size_t)s.rep * s.p.N : reinterpret_cast<uint32_t *>(sm + L.off_pfjob);
    s.K = reinterpret_cast<uint32_t *>(sm + L.off_K);
    s.Kpend = reinterpret_cast<uint32_t *>(sm + L.off_Kpend);
    s.ndec = reinterpret_cast<uint16_t *>(sm + L.off_ndec);
    s.nact = reinterpret_cast<uint16_t *>(sm + L.off_nact);
    s.pfcur = reinterpret_cast<uint16_t *>(sm + L.off_pfcur);
    s.sfin16 = reinterpret_cast<uint16_t *>(sm + L.off_sfin16);
    s.socc = reinterpret_cast<uint32_t *>(sm + L.off_socc);
    s.touch = reinterpret_cast<uint32_t *>(sm + L.off_touch);
    s.gate_xi = reinterpret_cast<double *>(sm + L.off_gate);
    s.gate_dq = s.gate_xi + MAXI;
    s.gate_ok = reinterpret_cast<uint32_t *>(s.gate_dq + MAXI);
    s.cs = reinterpret_cast<ClassState *>(sm + L.off_cs);
    s.aring = reinterpret_cast<ADraw *>(sm + L.off_ring);
    s.st_rec = reinterpret_cast<SlotRec *>(sm + L.off_strec);
    s.st_te = reinterpret_cast<double *>(sm + L.off_stte);
    s.pqh = reinterpret_cast<QEntry *>(sm + L.off_pqh);
    s.wcs = reinterpret_cast<WarpClassStats *>(sm + L.off_wcs);
    s.cmd = reinterpret_cast<MwCmd *>(sm + L.off_cmd);
    s.res = reinterpret_cast<MwRes *>(sm + L.off_res);
    s.n_pend = 0;
    s.rec_after = 0;
    s.ring_n = 0; s.ring_pos = 0; s.sched_pending = false; s.t0_pending = 0.0;
    const Params &p = s.p;
    const size_t r = s.rep;
    s.s_fin = p.slot_fin + r * (size_t)p.N * p.B;
    s.s_rec = p.slot_rec + r * (size_t)p.N * p.B;
    s.pq = p.pq + r * (size_t)p.I * p.qcap;
    s.dq = p.dq + r * (size_t)2 * p.qcap;
    s.hist = p.hist_mem ? p.hist_mem + r * (size_t)p.I * 2 * NBIN : nullptr;
}

// Empty system at t = 0: idle GPUs, first arrival of every class scheduled, abandonment levels drawn.
__global__ void __launch_bounds__(32) qsim_init_kernel(Params p)
{
    constexpr int SPLT = 0;
    constexpr uint32_t FT = F_GENERIC;
    extern __shared__ __align__(16) char sm[];
    const int lane = threadIdx.x;
    for (uint32_t rep = blockIdx.x; rep < p.R; rep += gridDim.x) {
        const SmemLayout L = smem_layout(p.Npad, p.B, p.slots_smem, 1, p.coef[5] != 0.0, p.tarr_global != 0, p.I);
        Sim<SPLT, FT> s(p, lane, rep);
        bind_pointers(s, sm, L);
        __syncwarp();
        for (uint32_t o = lane * 4; o < L.total; o += 128) *reinterpret_cast<uint32_t *>(sm + o) = 0;
        __syncwarp();
        for (uint32_t g = lane; g < p.Npad; g += 32) { s.tnext[g] = dinf(); s.nfin[g] = NONE32; }
        if (p.slots_smem && (p.B & 31u)) {
            const uint32_t bw = (p.B + 31u) >> 5;
            for (uint32_t g = lane; g < p.Npad; g += 32) s.socc[g * bw + bw - 1] = ~0u << (p.B & 31u);
        }
        if (p.tarr_global)
            for (uint32_t g = lane; g < p.N; g += 32) { s.pf_tarr[g] = 0.0; s.pfjob[g] = 0; }
        if (lane < (int)p.I) {
            ClassState &c = s.cs[lane];
            c.ta = dinf();
            AbClock *clk[3] = { &c.abp, &c.abd0, &c.abd1 };
            const uint32_t streams[3] = { STREAM_ABANDON_P, STREAM_ABANDON_D0, STREAM_ABANDON_D1 };
            for (int k = 0; k < 3; ++k) {
                uint32_t w0, w1, w2, w3;
                draw(p, rep, (streams[k] << 8) | (uint32_t)lane, 0, w0, w1, w2, w3);
                clk[k]->acc = 0.0; clk[k]->lvl = -qlog(u53(w0, w1)); clk[k]->t_last = 0.0; clk[k]->t_ab = dinf();
                clk[k]->m = 1;
            }
        }
        __syncwarp();
        // first arrival of every class: ask for draws, let the warp fill the rings, give the unused draws back
        s.sched_pending = lane < (int)p.I && p.n_inject == 0;
        s.t0_pending = 0.0;
        if (p.n_inject > 0 && lane < (int)p.I) s.schedule_from(0.0);
        for (int guard = 0; guard < 64; ++guard) {
            uint32_t need = __ballot_sync(FULL, s.sched_pending);
            if (!need) break;
            for (; need; need &= need - 1) s.refill((uint32_t)__ffs((int)need) - 1u);
        }
        if (lane < (int)p.I) s.cs[lane].adraw -= s.ring_n;
        __syncwarp();
        // write everything out
        RepHeader &h = p.hdr[rep];
        for (uint32_t o = lane * 4; o < sizeof(RepHeader); o += 128)
            *reinterpret_cast<uint32_t *>(reinterpret_cast<char *>(&h) + o) = 0;
        __syncwarp();
        if (lane < (int)p.I) h.cs[lane] = s.cs[lane];
        char *img = p.srv + (size_t)rep * p.srv_bytes;
        for (uint32_t o = lane * 16; o < L.srv_bytes; o += 512)
            *reinterpret_cast<uint4 *>(img + o) = *reinterpret_cast<const uint4 *>(sm + o);
        if (p.hist_mem)
            for (uint32_t o = lane; o < p.I * 2 * NBIN; o += 32) s.hist[o] = 0;
        __syncwarp();
    }
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *a)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *a, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(a), "r"(v) : "memory");
}
// A block waits this many times about a microsecond (minutes in all) for the chunk before its own before it gives up.
// Another block is running that chunk, so the wait lasts one chunk at most.
constexpr uint32_t CHUNK_SPIN_LIMIT = 1u << 28;

// Advance replications to their new end time (or until the per-launch event budget runs out).
template <int SPLT, uint32_t FT>
// One-warp instances whose slot records live in global memory need little shared memory, so registers decide how many
// replications are resident on an SM: they are compiled for at least 12 blocks per SM (at most 168 registers, a few
// bytes of spills; +16-24 % at N = 64 with thousands of replications).  Instances with the finish stamps on chip are
// limited by shared memory and keep all the registers they want (the cap cost them 13 %).
#ifndef QSIM_MIN_BLOCKS
#define QSIM_MIN_BLOCKS 12
#endif
__global__ void __launch_bounds__((FT & F_MW) ? 32 * MW_MAX : 32, ((FT & F_MW) || (FT & F_SLOTS)) ? 1 : QSIM_MIN_BLOCKS) qsim_run_kernel(Params p)
{
    extern __shared__ __align__(16) char sm[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t nthr = blockDim.x;
    // With nchunk = K > 1 the grid is one block per resident slot and the work is R x K units (chunk c of replication r is
    // unit c R + r), handed out in that order through a counter: replications outnumbering the slots then finish together
    // instead of leaving a last, nearly empty wave.  Chunk c of a replication starts when chunk c - 1 has published its
    // stamp; that unit was handed out earlier, so the block it waits for is running.  The chunks end at the times at
    // which K successive launches would end, so the result is theirs: that of one launch, up to the order in which the
    // fp64 sums of finished requests are added to the totals.
    __shared__ uint32_t sh_unit[2];
    const uint32_t K = p.nchunk > 1 ? p.nchunk : 1u;
    const uint32_t n_units = p.R * K;
    for (uint32_t unit = blockIdx.x;; unit += gridDim.x) {
        if (K > 1) {
            if (tid == 0) sh_unit[0] = atomicAdd(p.not_done + 1, 1u);
            if (FT & F_MW) __syncthreads(); else __syncwarp();
            unit = sh_unit[0];
            if (FT & F_MW) __syncthreads(); else __syncwarp();
        }
        if (unit >= n_units) break;
        const uint32_t rep = unit % p.R, chunk = unit / p.R;
        RepHeader &h = p.hdr[rep];
        uint32_t advance = p.advance, chunks_left = 0;
        unsigned long long horizon_iters = p.horizon_iters;
        if (K > 1) {
            if (tid == 0) {
                uint32_t ok = 1;
                if (chunk > 0) {
                    const uint32_t want = p.launch_tag + chunk;
                    for (uint32_t spins = 0; ld_acquire_u32(&h.seq) != want; ++spins) {
                        if (spins > CHUNK_SPIN_LIMIT || ld_acquire_u32(p.not_done + 2) != 0) { ok = 0; break; }
                        __nanosleep(1000);
                    }
                }
                sh_unit[1] = ok;
            }
            if (FT & F_MW) __syncthreads(); else __syncwarp();
            const uint32_t ok = sh_unit[1];
            __threadfence();
            if (FT & F_MW) __syncthreads(); else __syncwarp();
            if (!ok) {      // the chunk before this one did not finish in time: report, start nothing
                if (tid == 0) { atomicExch(p.not_done + 2, 1u); atomicAdd(p.not_done, 1u); }
                continue;
            }
            const bool first = chunk == 0 && p.advance == 1;
            chunks_left = first ? K : h.chunks_left;
            bool idle = false;
            if (!first && !h.done) advance = 0;                 // stopped on the event budget: go on to the same end time
            else if (chunks_left > 0) {
                const unsigned long long j = K - chunks_left;
                horizon_iters = p.horizon_iters * (j + 1) / K - p.horizon_iters * j / K;
                advance = 1;
                --chunks_left;
            } else idle = true;
            if (idle) {
                if (FT & F_MW) __syncthreads(); else __syncwarp();
                if (tid == 0) st_release_u32(&h.seq, p.launch_tag + chunk + 1u);
                continue;
            }
        } else if (!p.advance && h.done) continue;
        const SmemLayout L = smem_layout(p.Npad, p.B, p.slots_smem, nthr >> 5, p.coef[5] != 0.0, p.tarr_global != 0, p.I);
        Sim<SPLT, FT> s(p, lane, rep);
        s.warp = warp;
        s.nwarps = (int)(nthr >> 5);
        bind_pointers(s, sm, L);
        s.block_sync();
        // stage state: per-GPU arrays (coalesced 16-byte copies) and the class records; clear the per-warp accounting
        const char *img = p.srv + (size_t)rep * p.srv_bytes;
        for (uint32_t o = tid * 16; o < L.srv_bytes; o += nthr * 16)
            *reinterpret_cast<uint4 *>(sm + o) = *reinterpret_cast<const uint4 *>(img + o);
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(h.cs);
            uint4 *dst = reinterpret_cast<uint4 *>(s.cs);
            for (uint32_t o = tid; o < sizeof(ClassState) * p.I / 16; o += nthr) dst[o] = src[o];
            uint32_t *w = reinterpret_cast<uint32_t *>(s.wcs);
            for (uint32_t o = tid; o < sizeof(WarpClassStats) * MAXI * (nthr >> 5) / 4; o += nthr) w[o] = 0;
        }
        s.block_sync();
        // the end time is one rounded product of the cumulative horizon: run(a); run(b) ends where run(a+b) ends
        double T_end = h.T_end;
        const unsigned long long H_total = h.H_total + (advance == 1 ? horizon_iters : 0ull);
        if (advance == 1) T_end = __dmul_rn((double)H_total, iter_time(p, 0, p.B, 0));
        if (advance == 2) T_end = p.T_abs;
        s.T_end = T_end;
        s.T_reset = h.T_reset;
        s.tau_min = fmin(p.coef[0], p.coef[3]);
        s.t = 0.0;
        s.load_block(h.blk);
        s.dq_head0 = h.dq_head0; s.dq_head1 = h.dq_head1; s.dq_n0 = h.dq_n0; s.dq_n1 = h.dq_n1;
        s.place_ord = h.place_ord; s.events = h.events; s.rounds = h.rounds; s.sel_ord0 = h.sel_ord0; s.sel_ord1 = h.sel_ord1;
        s.n_touch = 0; s.touch_all = false; s.need_start = 0; s.err = h.err;
        s.drain_dirty = true; s.gate_dirty = true;
        s.force_nonlocal = (p.force_dispatch != 0 && chunk == 0) || h.force != 0;
        s.n_idle_pf = 0;
        s.idle_hint = NONE32;
        s.it_mixed = 0; s.it_solo = 0; s.busy_mixed = 0.0; s.busy_solo = 0.0;
        bool finished = true;
        if (warp == 0) {
            s.n_idle_pf = s.count_idle_pf();
            if (lane < (int)p.I && s.cs[lane].pq_n > 0) s.pqh[lane] = s.pq[(size_t)lane * p.qcap + s.cs[lane].pq_head];
            __syncwarp();
            s.it_mixed = h.iters_mixed[lane]; s.it_solo = h.iters_solo[lane];
            s.busy_mixed = h.busy_mixed[lane]; s.busy_solo = h.busy_solo[lane];
            finished = s.err ? true : s.run();
            s.flush_done();
            if (FT & F_MW) {
                if (lane == 0) s.cmd->op = MW_EXIT;
                __syncthreads();
            }
        } else {
            s.helper_loop();
        }
        s.block_sync();
        s.merge_warp_stats();
        if (warp == 0 && lane < (int)p.I) s.cs[lane].adraw -= s.ring_n;     // unused arrival draws are produced again next time
        s.block_sync();
        // stage back
        char *out = p.srv + (size_t)rep * p.srv_bytes;
        for (uint32_t o = tid * 16; o < L.srv_bytes; o += nthr * 16)
            *reinterpret_cast<uint4 *>(out + o) = *reinterpret_cast<const uint4 *>(sm + o);
        {
            uint4 *dst = reinterpret_cast<uint4 *>(h.cs);
            const uint4 *src = reinterpret_cast<const uint4 *>(s.cs);
            for (uint32_t o = tid; o < sizeof(ClassState) * p.I / 16; o += nthr) dst[o] = src[o];
        }
        // per-thread partial sums go to the 32 lane slots, warp after warp (a fixed order)
        for (int w = 0; w < s.nwarps; ++w) {
            if (warp == w) {
                if (w == 0) {
                    h.iters_mixed[lane] = s.it_mixed; h.iters_solo[lane] = s.it_solo;
                    h.busy_mixed[lane] = s.busy_mixed; h.busy_solo[lane] = s.busy_solo;
                } else {
                    h.iters_mixed[lane] += s.it_mixed; h.iters_solo[lane] += s.it_solo;
                    h.busy_mixed[lane] = __dadd_rn(h.busy_mixed[lane], s.busy_mixed);
                    h.busy_solo[lane] = __dadd_rn(h.busy_solo[lane], s.busy_solo);
                }
            }
            if (FT & F_MW) { __threadfence_block(); __syncthreads(); }
        }
        if (tid == 0) {
            h.T_end = T_end; h.H_total = H_total; h.blk = s.blk;
            h.dq_head0 = s.dq_head0; h.dq_head1 = s.dq_head1; h.dq_n0 = s.dq_n0; h.dq_n1 = s.dq_n1;
            h.place_ord = s.place_ord; h.events = s.events; h.rounds = s.rounds; h.err = s.err;
            h.sel_ord0 = s.sel_ord0; h.sel_ord1 = s.sel_ord1;
            h.done = finished ? 1u : 0u;
            h.force = s.force_nonlocal ? 1u : 0u;
            if (K > 1) {
                h.chunks_left = chunks_left;
                if (chunk == K - 1u && (!finished || chunks_left > 0)) atomicAdd(p.not_done, 1u);
            } else if (!finished) atomicAdd(p.not_done, 1u);
        }
        if (K > 1) {        // hand the replication over to the unit of its next chunk
            __threadfence();
            s.block_sync();
            if (tid == 0) st_release_u32(&h.seq, p.launch_tag + chunk + 1u);
        }
        s.block_sync();
    }
}

// Zero the statistics of every replication, keep the simulated state.
__global__ void qsim_reset_kernel(Params p)
{
    const uint32_t rep = blockIdx.x * blockDim.x + threadIdx.x;
    if (rep >= p.R) return;
    RepHeader &h = p.hdr[rep];
    const double T = h.T_end;
    h.T_reset = T;
    h.events = 0;
    h.rounds = 0;
    for (int l = 0; l < 32; ++l) { h.iters_mixed[l] = 0; h.iters_solo[l] = 0; h.busy_mixed[l] = 0.0; h.busy_solo[l] = 0.0; }
    for (uint32_t i = 0; i < MAXI; ++i) {
        ClassState &c = h.cs[i];
        Area *as[3] = { &c.aQp, &c.aX, &c.aQd };
        for (int k = 0; k < 3; ++k) { as[k]->area = 0.0; as[k]->t_last = T; }
        c.sYm_in = c.sYm_out = c.sYs_in = c.sYs_out = 0.0;
        c.arrivals = c.admitted = c.prefill_done = c.placed_mixed = c.placed_solo = c.done_mixed = c.done_solo = 0;
        c.abandoned_p = c.abandoned_d = c.overflow = c.overflow_d = c.tok_in_pf = c.tok_in_done = c.tok_out_done = 0;
        c.sum_ttft = 0.0; c.sum_tpot = 0.0;
    }
    if (p.hist_mem) {
        uint32_t *hm = p.hist_mem + (size_t)rep * p.I * 2 * NBIN;
        for (uint32_t o = 0; o < p.I * 2 * NBIN; ++o) hm[o] = 0;
    }
}

}  // namespace qsimdev
