// Device side of qsim, second kernel family: one thread simulates one replication.
//
// A replication is a strictly sequential chain of events.  The warp-per-replication kernels of qsim_device.cuh spend
// a whole warp on that chain; when there are thousands of replications it pays to give every replication one thread
// instead and let the 32 lanes of a warp advance 32 chains at once.  A lane then runs a plain event-driven simulation,
// event by event in the order (time, source id), with the dispatch (decode routing, prefill gate, iteration starts)
// after every event, exactly as the method is stated; what makes it fast is that no step looks at all GPUs:
//   * next iteration end: a calendar queue over the simulated GPUs (buckets of equal width in time, one bit per
//     non-empty bucket, GPUs of a bucket chained through their records); every pending end lies less than one
//     revolution ahead because an iteration is never longer than tau_max, so bucket order is time order;
//   * least-loaded GPU with a free decode slot (solo tier, mixed tier) and least-loaded mixed GPU with an idle prefill
//     slot: three 8-ary tournament trees over the keys (decodes << 16 | GPU), a leaf is NONE32 when the GPU is not
//     eligible; the root is the answer, an update reads one 32-byte group per level;
//   * decodes that emit their last token: per simulated GPU an 8-ary tournament tree over the finish iterations of its
//     B slots (keys finish << 16 | slot); the root is the GPU's next finish, a retirement recomputes one path.
// All state of a replication lives in global memory (its hot part stays in the caches); the lanes of a warp never
// communicate.  Clock arithmetic is the same chain of rounded IEEE operations as in the other family.
#pragma once

#include "qsim_device.cuh"

namespace qsimdev {

constexpr uint32_t NONE16 = 0xffffu;

// One simulated GPU: 32 bytes, one memory sector.
struct LaneSrv {
    double tnext;                 // end of the running iteration; +inf when the GPU is between iterations
    uint32_t it, nfin, pfjob;     // finished iterations; earliest finish iteration among its decodes; prefill request (bit 31 = present)
    uint16_t pfrem, pfcur, ndec, nact, cnext, ftop;  // prompt tokens left, chunk of the running iteration, decodes held, decodes in the
                                                     // running batch, next GPU in the same calendar bucket, the slot on top of the GPU's
                                                     // stack of free slots when it is known (NONE16 otherwise)
};
static_assert(sizeof(LaneSrv) == 32, "LaneSrv is one sector");

__device__ __forceinline__ unsigned long long dbits(double x) { return (unsigned long long)__double_as_longlong(x); }

__device__ __forceinline__ uint32_t min8(const uint32_t v[8])
{
    return min(min(min(v[0], v[1]), min(v[2], v[3])), min(min(v[4], v[5]), min(v[6], v[7])));
}

// LF = features compiled into an instance of the lane kernels: LF_GENERIC reads every mode from the parameters; otherwise the
// set bits say what the instance contains (abandonment, SLI-aware router, histograms, blocks) and the rest is compiled out.
constexpr uint32_t LF_GENERIC = 1, LF_ABANDON = 2, LF_SLI = 4, LF_HIST = 8, LF_BLOCKS = 16;

template <uint32_t LF>
struct LaneSim {
    const Params &p;
    const uint32_t rep;
    RepHeader &h;
    // this replication's arrays
    LaneSrv *srv;
    double *tarr;
    uint16_t *chead;
    uint32_t *cbm;               // the bitmap's home in global memory
    uint32_t *tsolo, *tmix, *tpf;
    uint32_t *sfin;
    unsigned long long *snode;
    SlotRec *srec;
    uint16_t *sfree;
    QEntry *pq, *dq;
    uint32_t *pql;               // [I][qw] one bit per prefill-queue position: the entry is a waiting request
    uint32_t *hist;
    // shared memory of this lane: class records (copied in at kernel entry, back at exit) and the calendar's bitmap
    // (word w of lane l at w * 32 + l)
    ClassState *cs;
    uint32_t *sbm;
    // one GPU record kept in registers across the steps of an event (the event's own GPU)
    uint32_t cg;
    LaneSrv crec;
    // scalars of the run
    double t, T_end, T_blk_next, T_reset;
    uint32_t blk, M, err;
    uint32_t dq_head0, dq_head1, dq_n0, dq_n1;
    uint32_t root_solo, root_mix, root_pf;      // roots of the three eligibility trees
    unsigned long long events, rounds, it_mixed, it_solo;
    double busy_mixed, busy_solo;
    // earliest pending iteration end (valid while nothing earlier can have been inserted)
    bool nx_valid;
    unsigned long long nx_t;
    uint32_t nx_g, nx_b, nx_prev;
    LaneSrv nx_rec;
    // earliest event of the class sources and the block boundary
    bool cl_valid;
    unsigned long long cl_t;
    uint32_t cl_s;
    // GPUs that were between iterations when this event gave them work
    uint32_t touch0, touch1, touch2, touch3;
    uint32_t n_touch;
    bool touch_all, drain_dirty, gate_dirty;

    __device__ LaneSim(const Params &p_, uint32_t rep_) : p(p_), rep(rep_), h(p_.hdr[rep_]) {}

    __device__ __forceinline__ bool f_abandon() const { return (LF & LF_GENERIC) ? p.any_theta != 0 : (LF & LF_ABANDON) != 0; }
    __device__ __forceinline__ bool f_sli() const { return (LF & LF_GENERIC) ? p.router == 1 : (LF & LF_SLI) != 0; }
    __device__ __forceinline__ bool f_blocks() const { return (LF & LF_GENERIC) ? p.nblk > 1 : (LF & LF_BLOCKS) != 0; }
    __device__ __forceinline__ bool f_hist() const { return (LF & LF_GENERIC) ? hist != nullptr : (LF & LF_HIST) != 0; }
    __device__ __forceinline__ double block_start(uint32_t b) const { return __dmul_rn((double)b, p.block_len); }

    __device__ __forceinline__ void bind()
    {
        const LanePar &q = p.lane;
        const size_t r = rep;
        srv = q.srv + r * p.N;
        tarr = q.tarr + r * p.N;
        chead = q.cal_head + r * q.nbk;
        cbm = q.cal_bm + r * (q.nbk >> 5);
        tsolo = q.tree + r * 3 * q.tsize;
        tmix = tsolo + q.tsize;
        tpf = tmix + q.tsize;
        sfin = q.sfin + r * (size_t)p.N * q.b8;
        snode = q.snode + r * (size_t)p.N * q.ssize;
        srec = q.srec + r * (size_t)p.N * p.B;
        sfree = q.sfree + r * (size_t)p.N * p.B;
        pq = p.pq + r * (size_t)p.I * p.qcap;
        pql = q.pql + r * (size_t)p.I * q.qw;
        dq = p.dq + r * (size_t)2 * p.qcap;
        hist = p.hist_mem ? p.hist_mem + r * (size_t)p.I * 2 * NBIN : nullptr;
    }

    __device__ __forceinline__ void load_block(uint32_t b)
    {
        blk = b;
        M = p.blocks[b].M;
        T_blk_next = (f_blocks() && b + 1 < p.nblk) ? block_start(b + 1) : dinf();
    }

    // --- eligibility trees (8-ary minimum trees over 32-bit keys) ------------------------------------
    // Set leaf g of a tree to key and recompute its ancestors; returns the new root.  The sibling groups of all levels
    // are read first (their addresses depend on g only), the path itself is carried in registers.
    __device__ __forceinline__ uint32_t tree_set(uint32_t *tr, uint32_t g, uint32_t key)
    {
        const LanePar &q = p.lane;
        tr[g] = key;
        uint32_t grp[4][8];
        uint32_t child = g;
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            if (l < (int)q.tlev) {
                const uint32_t base = q.toff[l] + (child & ~7u);
                const uint4 a = *reinterpret_cast<const uint4 *>(tr + base), b = *reinterpret_cast<const uint4 *>(tr + base + 4);
                grp[l][0] = a.x; grp[l][1] = a.y; grp[l][2] = a.z; grp[l][3] = a.w;
                grp[l][4] = b.x; grp[l][5] = b.y; grp[l][6] = b.z; grp[l][7] = b.w;
                child >>= 3;
            }
        }
        uint32_t cur = key;
        child = g;
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            if (l < (int)q.tlev) {
                uint32_t m = NONE32;
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j) m = min(m, j == (child & 7u) ? cur : grp[l][j]);
                cur = m;
                child >>= 3;
                tr[q.toff[l + 1] + child] = cur;
            }
        }
        return cur;
    }

    // keys of GPU g in the three trees for nd decodes held and prefill presence pf
    __device__ __forceinline__ void keys_of(uint32_t g, uint32_t nd, bool pf, uint32_t &ks, uint32_t &km, uint32_t &kp) const
    {
        const bool mix = g < M;
        const uint32_t cap = (mix || pf) ? p.B - 1 : p.B;        // a mixed GPU keeps one slot for prefill (Eq. (13)-(14))
        const uint32_t key = (nd << 16) | g;
        ks = (!mix && nd < cap) ? key : NONE32;
        km = (mix && nd < cap) ? key : NONE32;
        kp = (mix && !pf && nd <= p.B - 1) ? key : NONE32;
    }

    // GPU g went from (nd0, pf0) to (nd1, pf1): update the trees whose leaf changed
    __device__ __forceinline__ void retree(uint32_t g, uint32_t nd0, bool pf0, uint32_t nd1, bool pf1)
    {
        uint32_t s0, m0, p0, s1, m1, p1;
        keys_of(g, nd0, pf0, s0, m0, p0);
        keys_of(g, nd1, pf1, s1, m1, p1);
        // a GPU is a leaf of the solo tree or of the mixed tree, never of both: one update serves either
        const bool mix = g < M;
        if (mix ? m0 != m1 : s0 != s1) {
            const uint32_t root = tree_set(mix ? tmix : tsolo, g, mix ? m1 : s1);
            if (mix) root_mix = root; else root_solo = root;
        }
        if (p0 != p1) root_pf = tree_set(tpf, g, p1);
    }

    // all three trees from the GPU records (at a change of M, and when a fresh state is first run)
    __device__ __forceinline__ void rebuild_trees()
    {
        const LanePar &q = p.lane;
        for (uint32_t g = 0; g < q.toff[1]; ++g) {
            uint32_t ks = NONE32, km = NONE32, kp = NONE32;
            if (g < p.N) {
                const LaneSrv s = srv[g];
                keys_of(g, s.ndec, (s.pfjob >> 31) != 0, ks, km, kp);
            }
            tsolo[g] = ks; tmix[g] = km; tpf[g] = kp;
        }
        for (uint32_t l = 0; l < q.tlev; ++l) {
            const uint32_t n_child = q.toff[l + 1] - q.toff[l], n_par = (l + 1 < q.tlev ? q.toff[l + 2] : q.tsize) - q.toff[l + 1];
            for (uint32_t k = 0; k < n_par; ++k) {
                uint32_t a = NONE32, b = NONE32, c = NONE32;
                if (k * 8 < n_child)
                    for (uint32_t j = 0; j < 8; ++j) {
                        const uint32_t o = q.toff[l] + k * 8 + j;
                        a = min(a, tsolo[o]); b = min(b, tmix[o]); c = min(c, tpf[o]);
                    }
                tsolo[q.toff[l + 1] + k] = a; tmix[q.toff[l + 1] + k] = b; tpf[q.toff[l + 1] + k] = c;
            }
        }
        root_solo = tsolo[q.toff[q.tlev]]; root_mix = tmix[q.toff[q.tlev]]; root_pf = tpf[q.toff[q.tlev]];
    }

    // --- decode slots of one GPU (8-ary minimum tree over finish << 16 | slot) ------------------------
    __device__ __forceinline__ void slot_insert(uint32_t g, uint32_t slot, uint32_t fin)
    {
        const LanePar &q = p.lane;
        sfin[(size_t)g * q.b8 + slot] = fin;
        unsigned long long *nd = snode + (size_t)g * q.ssize;
        const unsigned long long key = ((unsigned long long)fin << 16) | slot;
        unsigned long long old[4];
        uint32_t child = slot;
#pragma unroll
        for (int l = 0; l < 4; ++l)
            if (l < (int)q.slev) { child >>= 3; old[l] = nd[q.soff[l] + child]; }
        child = slot;
#pragma unroll
        for (int l = 0; l < 4; ++l)
            if (l < (int)q.slev) { child >>= 3; if (key < old[l]) nd[q.soff[l] + child] = key; }
    }

    // free the slot and recompute its path; returns the new root (finish << 16 | slot, all ones when the GPU holds no decode)
    __device__ __forceinline__ unsigned long long slot_remove(uint32_t g, uint32_t slot)
    {
        const LanePar &q = p.lane;
        uint32_t *leaf = sfin + (size_t)g * q.b8;
        unsigned long long *nd = snode + (size_t)g * q.ssize;
        const unsigned long long INF64 = ~0ull;
        const uint32_t base = slot & ~7u;
        const uint4 a = *reinterpret_cast<const uint4 *>(leaf + base), b = *reinterpret_cast<const uint4 *>(leaf + base + 4);
        const uint32_t lf[8] = { a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w };
        unsigned long long grp[3][8];
        uint32_t child = slot >> 3;
#pragma unroll
        for (int l = 1; l < 4; ++l) {
            if (l < (int)q.slev) {
                const unsigned long long *src = nd + q.soff[l - 1] + (child & ~7u);
#pragma unroll
                for (uint32_t j = 0; j < 8; j += 2) {
                    const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(src + j);
                    grp[l - 1][j] = v.x; grp[l - 1][j + 1] = v.y;
                }
                child >>= 3;
            }
        }
        leaf[slot] = NONE32;
        unsigned long long cur = INF64;
#pragma unroll
        for (uint32_t j = 0; j < 8; ++j) {
            const unsigned long long k = (lf[j] == NONE32 || j == (slot & 7u)) ? INF64 : (((unsigned long long)lf[j] << 16) | (base + j));
            cur = k < cur ? k : cur;
        }
        child = slot >> 3;
        nd[q.soff[0] + child] = cur;
#pragma unroll
        for (int l = 1; l < 4; ++l) {
            if (l < (int)q.slev) {
                unsigned long long m = INF64;
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j) {
                    const unsigned long long k = j == (child & 7u) ? cur : grp[l - 1][j];
                    m = k < m ? k : m;
                }
                cur = m;
                child >>= 3;
                nd[q.soff[l] + child] = cur;
            }
        }
        return cur;
    }

    // --- GPU records -------------------------------------------------------------------------------------
    __device__ __forceinline__ LaneSrv load_srv(uint32_t g) const { return g == cg ? crec : srv[g]; }
    __device__ __forceinline__ void store_srv(uint32_t g, const LaneSrv &s) { if (g == cg) crec = s; else srv[g] = s; }
    __device__ __forceinline__ void cache_flush() { if (cg != NONE32) { srv[cg] = crec; cg = NONE32; } }

    // --- calendar of iteration ends ---------------------------------------------------------------------
    __device__ __forceinline__ uint32_t &bm(uint32_t w) const { return sbm[(w << p.lane.lsh)]; }
    __device__ __forceinline__ uint32_t bucket_of(double x) const
    {
        return (uint32_t)__double2ull_rd(__dmul_rn(x, p.lane.inv_w)) & (p.lane.nbk - 1u);
    }

    // earliest pending iteration end: first non-empty bucket at or after the bucket of the current time, then the
    // earliest (time, GPU) of its chain
    __device__ __forceinline__ void peek()
    {
        const unsigned long long INF = 0x7ff0000000000000ull;
        const uint32_t W = p.lane.nbk >> 5;
        const uint32_t cb = bucket_of(t), wi = cb >> 5;
        uint32_t w = bm(wi) & (~0u << (cb & 31u));
        uint32_t k = 0;
        while (!w && k < W) {
            ++k;
            w = bm((wi + k) & (W - 1u));
            if (k == W) w &= ~(~0u << (cb & 31u));      // back at the first word: the buckets before the current one
        }
        nx_valid = true;
        if (!w) { nx_t = INF; nx_g = NONE32; return; }
        const uint32_t b = (((wi + k) & (W - 1u)) << 5) + (uint32_t)__ffs((int)w) - 1u;
        nx_b = b;
        nx_t = INF; nx_g = NONE32; nx_prev = NONE32;
        uint32_t cur = chead[b], prev = NONE32;
        for (uint32_t guard = 0; cur != NONE16 && guard <= p.N; ++guard) {
            const LaneSrv s = srv[cur];
            const unsigned long long v = dbits(s.tnext);
            if (v < nx_t || (v == nx_t && cur < nx_g)) { nx_t = v; nx_g = cur; nx_prev = prev; nx_rec = s; }
            prev = cur;
            cur = s.cnext;
        }
        if (nx_g == NONE32) err = ERR_INTERNAL;
    }

    // take the GPU found by peek out of its bucket
    __device__ __forceinline__ void pop_next()
    {
        const uint32_t nxt = nx_rec.cnext;
        if (nx_prev == NONE32) {
            chead[nx_b] = (uint16_t)nxt;
            if (nxt == NONE16) bm(nx_b >> 5) &= ~(1u << (nx_b & 31u));
        } else {
            srv[nx_prev].cnext = (uint16_t)nxt;
        }
        nx_valid = false;
    }

    // GPU g (record s, about to be written by the caller) starts an iteration that ends at s.tnext
    __device__ __forceinline__ void calendar_insert(uint32_t g, LaneSrv &s)
    {
        const uint32_t b = bucket_of(s.tnext);
        const uint32_t word = bm(b >> 5), bit = 1u << (b & 31u);
        uint32_t nxt = NONE16;
        if (word & bit) nxt = chead[b];
        else bm(b >> 5) = word | bit;
        s.cnext = (uint16_t)nxt;
        chead[b] = (uint16_t)g;
        if (nx_valid) {
            const unsigned long long v = dbits(s.tnext);
            if (b == nx_b || v < nx_t || (v == nx_t && g < nx_g)) nx_valid = false;
        }
    }

    // --- arrivals -----------------------------------------------------------------------------------------
    // Next arrival of class i after t0.  A candidate at or past the end of its block is discarded and drawn again from
    // the boundary under the next block's rate (memorylessness).
    __device__ __forceinline__ void schedule_arrival(uint32_t i, double t0)
    {
        ClassState &c = cs[i];
        uint32_t b = c.ablk;
        for (uint32_t guard = 0; guard < 4096; ++guard) {
            const double Lam = __dmul_rn((double)p.N, p.blocks[b].rate[i]);
            const bool has_next = f_blocks() && b + 1 < p.nblk;
            if (!(Lam > 0.0)) {
                if (!has_next) { c.ta = dinf(); c.ablk = b; return; }
                ++b; t0 = block_start(b);
                continue;
            }
            const ADraw d = make_draw(p.seed, p.rep_offset + rep, i, p.I, c.adraw, p.length_mode == 1 ? p.lengths : nullptr,
                                      p.cls[i].P, p.cls[i].D, 0.0);
            c.adraw++;
            const double cand = __dadd_rn(t0, __ddiv_rn(d.E, Lam));
            if (has_next && cand >= block_start(b + 1)) {
                ++b; t0 = block_start(b);
                continue;
            }
            c.ta = cand; c.ablk = b; c.nextP = job_P(d.pk); c.nextD = job_D(d.pk);
            return;
        }
        err = ERR_INTERNAL;
    }

    __device__ __forceinline__ void on_arrival(uint32_t i)
    {
        ClassState &c = cs[i];
        c.arrivals++;
        if (c.pq_n >= p.qcap) {
            c.overflow++;
        } else {
            if (f_abandon()) ab_change(c.abp, p.cls[i].theta, c.pq_n, c.pq_n + 1, t);
            area_touch(c.aQp, c.pq_n, t);
            if (c.pq_n == 0) { c.pq_head = 0; c.pq_tail = 0; }
            else if (c.pq_tail == c.pq_head) pq_compact(i);        // requests that left from inside the queue still hold positions
            const uint32_t pos = c.pq_tail;
            c.pq_tail = pos + 1 == p.qcap ? 0 : pos + 1;
            QEntry e; e.t = t; e.pk = pack_job(c.nextP, c.nextD, i, 0); e.cls = i;
            pq[(size_t)i * p.qcap + pos] = e;
            pql[(size_t)i * p.lane.qw + (pos >> 5)] |= 1u << (pos & 31u);
            c.pq_n++;
        }
        schedule_arrival(i, t);
        gate_dirty = true;
    }

    // --- prefill queues -----------------------------------------------------------------------------------
    // A class queue is a ring of qcap positions between pq_head (a waiting request whenever the queue is not empty) and
    // pq_tail, with one bit per position that says whether the entry still waits: a request that abandons from inside
    // the queue clears its bit and nothing moves.
    // Position of the r-th waiting request (r = 0: the first) at or after position `from`, in ring order.
    __device__ __forceinline__ uint32_t pq_find(uint32_t i, uint32_t from, uint32_t r)
    {
        const uint32_t *bits = pql + (size_t)i * p.lane.qw;
        const uint32_t nch = p.lane.qw >> 2;
        uint32_t c = from >> 7;
        for (uint32_t k = 0; k <= nch; ++k) {
            const uint4 v = *reinterpret_cast<const uint4 *>(bits + 4u * c);
            uint32_t w[4] = { v.x, v.y, v.z, v.w };
            if (k == 0 || k == nch) {
                // the chunk that holds `from`: positions from `from` on at the first visit, the ones before it at the last
#pragma unroll
                for (uint32_t j = 0; j < 4; ++j) {
                    const uint32_t base = (c << 7) + (j << 5);
                    const uint32_t below = from >= base + 32u ? ~0u : (from <= base ? 0u : ((1u << (from - base)) - 1u));
                    w[j] &= k == 0 ? ~below : below;
                }
            }
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) {
                const uint32_t n = (uint32_t)__popc(w[j]);
                if (r < n) return (c << 7) + (j << 5) + (uint32_t)__fns(w[j], 0, (int)r + 1);
                r -= n;
            }
            c = c + 1 == nch ? 0 : c + 1;
        }
        err = ERR_INTERNAL;
        return from;
    }

    // The waiting request at position pos of class i's queue (n requests wait) leaves it, by admission or abandonment.
    __device__ __forceinline__ void pq_take(uint32_t i, uint32_t pos, uint32_t n)
    {
        ClassState &c = cs[i];
        pql[(size_t)i * p.lane.qw + (pos >> 5)] &= ~(1u << (pos & 31u));
        if (pos == c.pq_head && n > 1) c.pq_head = pq_find(i, pos + 1 == p.qcap ? 0 : pos + 1, 0);
    }

    // Every position is taken although fewer than qcap requests wait: move the waiting ones together (rare).
    __device__ __forceinline__ void pq_compact(uint32_t i)
    {
        ClassState &c = cs[i];
        QEntry *ring = pq + (size_t)i * p.qcap;
        uint32_t *bits = pql + (size_t)i * p.lane.qw;
        uint32_t wr = c.pq_head, pos = c.pq_head;
        for (uint32_t k = 0; k < p.qcap; ++k) {
            if ((bits[pos >> 5] >> (pos & 31u)) & 1u) {
                if (pos != wr) {
                    ring[wr] = ring[pos];
                    bits[pos >> 5] &= ~(1u << (pos & 31u));
                    bits[wr >> 5] |= 1u << (wr & 31u);
                }
                wr = wr + 1 == p.qcap ? 0 : wr + 1;
            }
            pos = pos + 1 == p.qcap ? 0 : pos + 1;
        }
        c.pq_tail = wr;
    }

    // --- abandonment ----------------------------------------------------------------------------------------
    // remove entry pos (offset from head) of a ring of n entries, keeping the order
    __device__ __forceinline__ void ring_remove(QEntry *ring, uint32_t head, uint32_t n, uint32_t pos)
    {
        const uint32_t cap = p.qcap;
        for (uint32_t k = pos; k + 1 < n; ++k) {
            uint32_t src = head + k + 1; if (src >= cap) src -= cap;
            uint32_t dst = head + k; if (dst >= cap) dst -= cap;
            ring[dst] = ring[src];
        }
    }

    __device__ __forceinline__ void on_abandon_p(uint32_t i)
    {
        ClassState &c = cs[i];
        const uint32_t Q = c.pq_n;
        uint32_t w0, w1, w2, w3;
        draw(p, rep, (STREAM_ABANDON_P << 8) | i, c.abp.m, w0, w1, w2, w3);
        const uint32_t rank = __umulhi(w2, Q);       // uniformly chosen waiting request, in FCFS rank
        pq_take(i, pq_find(i, c.pq_head, rank), Q);
        area_touch(c.aQp, Q, t);
        c.pq_n = Q - 1;
        c.abandoned_p++;
        AbClock &a = c.abp;
        a.m++; a.acc = 0.0; a.lvl = -qlog(u53(w0, w1)); a.t_last = t;
        a.t_ab = (Q - 1 > 0) ? __dadd_rn(t, __ddiv_rn(a.lvl, __dmul_rn(p.cls[i].theta, (double)(Q - 1)))) : dinf();
    }

    __device__ __forceinline__ void on_abandon_d(uint32_t pool, uint32_t i)
    {
        ClassState &c = cs[i];
        const uint32_t Q = pool ? c.Qd1 : c.Qd0;
        AbClock &a = pool ? c.abd1 : c.abd0;
        uint32_t w0, w1, w2, w3;
        draw(p, rep, ((pool ? STREAM_ABANDON_D1 : STREAM_ABANDON_D0) << 8) | i, a.m, w0, w1, w2, w3);
        uint32_t rank = __umulhi(w2, Q);
        QEntry *ring = dq + (size_t)pool * p.qcap;
        const uint32_t head = (pool ? dq_head1 : dq_head0), n = (pool ? dq_n1 : dq_n0);
        uint32_t pos = NONE32;
        for (uint32_t k = 0; k < n; ++k) {
            uint32_t src = head + k; if (src >= p.qcap) src -= p.qcap;
            if (ring[src].cls == i) {
                if (rank == 0) { pos = k; break; }
                --rank;
            }
        }
        if (pos == NONE32) { err = ERR_INTERNAL; return; }
        ring_remove(ring, head, n, pos);
        (pool ? dq_n1 : dq_n0)--;
        area_touch(c.aQd, c.Qd0 + c.Qd1, t);
        if (pool) c.Qd1 = Q - 1; else c.Qd0 = Q - 1;
        c.abandoned_d++;
        a.m++; a.acc = 0.0; a.lvl = -qlog(u53(w0, w1)); a.t_last = t;
        a.t_ab = (Q - 1 > 0) ? __dadd_rn(t, __ddiv_rn(a.lvl, __dmul_rn(p.cls[i].theta, (double)(Q - 1)))) : dinf();
    }

    // --- end of an iteration on the GPU found by peek --------------------------------------------------------
    __device__ __forceinline__ void touch_gpu(uint32_t g)
    {
        if (n_touch == 0) touch0 = g; else if (n_touch == 1) touch1 = g; else if (n_touch == 2) touch2 = g; else if (n_touch == 3) touch3 = g;
        else touch_all = true;
        if (n_touch < 4) ++n_touch;
    }

    __device__ __forceinline__ void on_server()
    {
        const uint32_t g = nx_g;
        LaneSrv s = nx_rec;
        pop_next();
        const uint32_t itg = s.it + 1u, na = s.nact, pc = s.pfcur, nd0 = s.ndec;
        const bool pf0 = (s.pfjob >> 31) != 0;
        const double tau = iter_time(p, pc, na, 0, false);       // duration of the iteration that ends (same chain as at its start)
        if (pc > 0) { it_mixed++; busy_mixed = __dadd_rn(busy_mixed, tau); }
        else        { it_solo++;  busy_solo = __dadd_rn(busy_solo, tau); }
        s.it = itg;
        s.tnext = dinf();
        uint32_t nd = nd0;
        if (s.nfin == itg) {
            // every decode whose finish iteration is this one leaves: accounting, slot freed, next finish from the tree
            const LanePar &q = p.lane;
            unsigned long long root = snode[(size_t)g * q.ssize + q.soff[q.slev - 1]];
            for (uint32_t guard = 0; (uint32_t)(root >> 16) == itg && guard <= p.B; ++guard) {
                const uint32_t slot = (uint32_t)root & 0xffffu;
                const SlotRec r = srec[(size_t)g * p.B + slot];
                root = slot_remove(g, slot);
                --nd;
                sfree[(size_t)g * p.B + nd] = (uint16_t)slot;
                s.ftop = (uint16_t)slot;
                const uint32_t i = job_cls(r.pk), P = job_P(r.pk), D = job_D(r.pk);
                ClassState &c = cs[i];
                const double rel = __dsub_rn(t, T_reset);
                if (job_flag(r.pk)) { c.sYm_out = __dadd_rn(c.sYm_out, rel); c.Ym--; c.done_mixed++; }
                else                { c.sYs_out = __dadd_rn(c.sYs_out, rel); c.Ys--; c.done_solo++; }
                c.tok_in_done += P;        // bundled charging credits the request here, Eq. (21)-(22)
                c.tok_out_done += D;
                const double tpot = __ddiv_rn(__dsub_rn(t, r.tpf), (double)D);
                c.sum_tpot = __dadd_rn(c.sum_tpot, tpot);
                if (f_hist()) atomicAdd(&hist[((size_t)i * 2 + 1) * NBIN + hist_bin(tpot)], 1u);
            }
            s.nfin = (uint32_t)(root >> 16);
            s.ndec = (uint16_t)nd;
            drain_dirty = true;
            gate_dirty = true;
        }
        bool pf1 = pf0;
        if (pc > 0) {
            const uint32_t rem = (uint32_t)s.pfrem - pc;
            s.pfrem = (uint16_t)rem;
            if (rem == 0) {
                // prefill finished: account, then hand the request to the decode stage (it joins its pool's buffer)
                const uint32_t pk = s.pfjob;
                const uint32_t i = job_cls(pk), P = job_P(pk), D = job_D(pk);
                ClassState &c = cs[i];
                area_touch(c.aX, c.X, t);
                c.X--;
                c.prefill_done++;
                c.tok_in_pf += P;                  // separate charging credits the prompt here, Eq. (23)
                const double ttft = __dsub_rn(t, tarr[g]);
                c.sum_ttft = __dadd_rn(c.sum_ttft, ttft);
                if (f_hist()) atomicAdd(&hist[((size_t)i * 2 + 0) * NBIN + hist_bin(ttft)], 1u);
                uint32_t pool = 0;
                if (f_sli()) {
                    // SLI-aware router: one uniform per finished prefill decides the pool
                    uint32_t w0, w1, w2, w3;
                    draw(p, rep, (STREAM_SLI << 8) | i, c.sli_ord, w0, w1, w2, w3);
                    c.sli_ord++;
                    pool = (u53(w0, w1) <= p.blocks[blk].ps[i]) ? 0u : 1u;
                }
                s.pfjob = 0;
                pf1 = false;
                cl_valid = false;        // the buffer's abandonment clock moves
                if ((pool ? dq_n1 : dq_n0) >= p.qcap) {
                    c.overflow_d++;
                } else {
                    const uint32_t Qd = pool ? c.Qd1 : c.Qd0;
                    if (f_abandon()) ab_change(pool ? c.abd1 : c.abd0, p.cls[i].theta, Qd, Qd + 1, t);
                    area_touch(c.aQd, c.Qd0 + c.Qd1, t);
                    if (pool) c.Qd1++; else c.Qd0++;
                    uint32_t pos = (pool ? dq_head1 : dq_head0) + (pool ? dq_n1 : dq_n0);
                    if (pos >= p.qcap) pos -= p.qcap;
                    QEntry e; e.t = t; e.pk = pack_job(P, D, i, 0); e.cls = i;
                    dq[(size_t)pool * p.qcap + pos] = e;
                    (pool ? dq_n1 : dq_n0)++;
                }
                drain_dirty = true;
                gate_dirty = true;
            }
        }
        s.pfcur = 0;
        cg = g;                 // the record stays in registers until the event's dispatch has started the GPU again
        crec = s;
        if (nd != nd0 || pf1 != pf0) retree(g, nd0, pf0, nd, pf1);
        touch_gpu(g);
    }

    // An iteration end that changes nothing outside its GPU (no decode finishes, the prefill does not finish): the GPU
    // carries on with the same batch less one chunk.  Nothing is placed, admitted or freed, so no dispatch is needed.
    __device__ __forceinline__ bool end_is_plain(const LaneSrv &s) const
    {
        return s.nfin != s.it + 1u && !(s.pfcur > 0 && s.pfrem == s.pfcur);
    }

    __device__ __forceinline__ void plain_end()
    {
        const uint32_t g = nx_g;
        LaneSrv s = nx_rec;
        pop_next();
        const uint32_t pc = s.pfcur;
        const double tau = iter_time(p, pc, s.nact, 0, false);
        if (pc > 0) { it_mixed++; busy_mixed = __dadd_rn(busy_mixed, tau); s.pfrem = (uint16_t)(s.pfrem - pc); }
        else        { it_solo++;  busy_solo = __dadd_rn(busy_solo, tau); }
        s.it++;
        const uint32_t pc2 = (s.pfjob >> 31) ? min(p.C, (uint32_t)s.pfrem) : 0u;
        s.pfcur = (uint16_t)pc2;
        s.nact = s.ndec;          // requests placed meanwhile join here
        s.tnext = __dadd_rn(t, iter_time(p, pc2, s.ndec, 0, false));
        calendar_insert(g, s);
        srv[g] = s;
    }

    // --- dispatch ------------------------------------------------------------------------------------------------
    // head of the pool's buffer starts decoding on GPU g
    __device__ __forceinline__ void place_decode(uint32_t pool, uint32_t g)
    {
        const uint32_t head = (pool ? dq_head1 : dq_head0);
        const QEntry e = dq[(size_t)pool * p.qcap + head];
        LaneSrv s = load_srv(g);
        (pool ? dq_head1 : dq_head0) = (head + 1 == p.qcap) ? 0 : head + 1;
        (pool ? dq_n1 : dq_n0)--;
        const uint32_t i = e.cls, D = job_D(e.pk), P = job_P(e.pk);
        const bool mixed = g < M;
        ClassState &c = cs[i];
        cl_valid = false;            // the buffer's abandonment clock moves
        const uint32_t Qd = pool ? c.Qd1 : c.Qd0;
        if (f_abandon()) ab_change(pool ? c.abd1 : c.abd0, p.cls[i].theta, Qd, Qd - 1, t);
        area_touch(c.aQd, c.Qd0 + c.Qd1, t);
        if (pool) c.Qd1--; else c.Qd0--;
        const double rel = __dsub_rn(t, T_reset);
        if (mixed) { c.sYm_in = __dadd_rn(c.sYm_in, rel); c.Ym++; c.placed_mixed++; }
        else       { c.sYs_in = __dadd_rn(c.sYs_in, rel); c.Ys++; c.placed_solo++; }
        const uint32_t nd0 = s.ndec;
        const bool running = s.tnext < dinf(), pf = (s.pfjob >> 31) != 0;
        uint32_t slot = s.ftop;           // the top of the free-slot stack is known right after a retirement
        if (slot == NONE16) slot = sfree[(size_t)g * p.B + nd0];
        s.ftop = (uint16_t)NONE16;
        // joins the iteration that starts next: a running iteration first finishes as it+1
        const uint32_t fin = s.it + (running ? 1u : 0u) + D;
        SlotRec r; r.tpf = e.t; r.pk = pack_job(P, D, i, mixed ? 1u : 0u); r.pad = 0;
        srec[(size_t)g * p.B + slot] = r;
        slot_insert(g, slot, fin);
        s.ndec = (uint16_t)(nd0 + 1);
        s.nfin = min(s.nfin, fin);
        store_srv(g, s);
        if (nx_valid && nx_g == g) nx_rec = s;
        retree(g, nd0, pf, nd0 + 1, pf);
        if (!running) touch_gpu(g);
    }

    // Prefill gate: which waiting class goes next (occupancy gate of Section 4.1, priority gate of Section 5.1.1, or the
    // oldest head-of-line request of the FCFS ablation)
    __device__ __forceinline__ uint32_t gate_class()
    {
        uint32_t best = NONE32;
        if (p.gate == 2) {
            double bt = 0.0;
            for (uint32_t i = 0; i < p.I; ++i) {
                const ClassState &c = cs[i];
                if (c.pq_n == 0) continue;
                const double ta = pq[(size_t)i * p.qcap + c.pq_head].t;
                if (best == NONE32 || ta < bt) { best = i; bt = ta; }
            }
            return best;
        }
        if (p.gate == 1) {
            uint32_t key = NONE32;
            for (uint32_t i = 0; i < p.I; ++i)
                if (cs[i].pq_n > 0) key = min(key, (p.cls[i].prio << 8) | i);
            return key == NONE32 ? NONE32 : (key & 0xffu);
        }
        const BlockPar &bp = p.blocks[blk];
        double bxi = 0.0, bdq = 0.0;
        for (uint32_t i = 0; i < p.I; ++i) {
            const ClassState &c = cs[i];
            if (c.pq_n == 0 || !(bp.xstar[i] > 0.0)) continue;
            const double xi = __ddiv_rn(__dsub_rn((double)c.X, bp.nx[i]), bp.xstar[i]);   // xi_i = (X_i - n x*_i)/x*_i
            const double dqv = __dsub_rn((double)c.pq_n, bp.nq[i]);                         // Q_p,i - n q*_p,i
            if (best == NONE32 || xi < bxi || (xi == bxi && dqv > bdq)) { best = i; bxi = xi; bdq = dqv; }
        }
        return best;
    }

    __device__ __forceinline__ void admit(uint32_t i, uint32_t g)
    {
        ClassState &c = cs[i];
        const uint32_t head = c.pq_head;
        const QEntry e = pq[(size_t)i * p.qcap + head];
        LaneSrv s = load_srv(g);
        cl_valid = false;            // the queue's abandonment clock moves
        if (f_abandon()) ab_change(c.abp, p.cls[i].theta, c.pq_n, c.pq_n - 1, t);
        area_touch(c.aQp, c.pq_n, t);
        pq_take(i, head, c.pq_n);
        c.pq_n--;
        area_touch(c.aX, c.X, t);
        c.X++;
        c.admitted++;
        s.pfjob = e.pk | 0x80000000u;
        s.pfrem = (uint16_t)job_P(e.pk);
        tarr[g] = e.t;
        store_srv(g, s);
        if (nx_valid && nx_g == g) nx_rec = s;
        retree(g, s.ndec, false, s.ndec, true);
        if (!(s.tnext < dinf())) touch_gpu(g);
    }

    // A GPU with work that is between iterations starts one now: the batch (prefill chunk, decodes) is frozen here.
    __device__ __forceinline__ void start_gpu(uint32_t g)
    {
        LaneSrv s = load_srv(g);
        const bool has_pf = (s.pfjob >> 31) != 0;
        if (s.tnext < dinf() || (s.ndec == 0 && !has_pf)) return;
        const uint32_t pc = has_pf ? min(p.C, (uint32_t)s.pfrem) : 0u;
        s.pfcur = (uint16_t)pc;
        s.nact = s.ndec;
        s.tnext = __dadd_rn(t, iter_time(p, pc, s.ndec, 0, false));
        calendar_insert(g, s);
        store_srv(g, s);
    }

    __device__ __forceinline__ void dispatch()
    {
        // decode routing: buffered requests first (FCFS), solo GPUs before mixed ones; under the SLI-aware router the solo
        // pool's buffer feeds the solo GPUs and the mixed pool's buffer the mixed GPUs
        if (drain_dirty) {
            for (uint32_t guard = 0; guard <= 2u * p.qcap; ++guard) {
                uint32_t pool = 0, key = NONE32;
                if (!f_sli()) {
                    if (dq_n0 > 0) key = root_solo != NONE32 ? root_solo : root_mix;
                } else if (dq_n0 > 0 && root_solo != NONE32) {
                    key = root_solo;
                } else if (dq_n1 > 0 && root_mix != NONE32) {
                    pool = 1; key = root_mix;
                }
                if (key == NONE32) break;
                place_decode(pool, key & 0xffffu);
            }
        }
        drain_dirty = false;
        // prefill gate on the mixed GPUs whose prefill slot is idle
        if (gate_dirty) {
            while (root_pf != NONE32) {
                const uint32_t i = gate_class();
                if (i == NONE32) break;
                admit(i, root_pf & 0xffffu);
            }
        }
        gate_dirty = false;
        // every GPU that got work while it was between iterations starts its next iteration now
        {
            const uint32_t n = touch_all ? p.N : n_touch;
            for (uint32_t k = 0; k < n; ++k) start_gpu(touch_all ? k : (k == 0 ? touch0 : (k == 1 ? touch1 : (k == 2 ? touch2 : touch3))));
        }
        n_touch = 0;
        touch_all = false;
        cache_flush();
    }

    // --- the event loop ----------------------------------------------------------------------------------------
    // earliest event among the block boundary and the class clocks; sources are scanned in id order with '<', which
    // keeps the tie order (block end, arrivals, prefill-queue abandonments, decode-buffer abandonments by pool)
    __device__ __forceinline__ void class_candidates()
    {
        const unsigned long long INF = 0x7ff0000000000000ull;
        unsigned long long bt = INF;
        uint32_t bs = NONE32;
        if (f_blocks() && T_blk_next < dinf()) { bt = dbits(T_blk_next); bs = SRC_BLOCK; }
        for (uint32_t i = 0; i < p.I; ++i) { const unsigned long long v = dbits(cs[i].ta); if (v < bt) { bt = v; bs = SRC_ARRIVAL + i; } }
        if (f_abandon()) {
            for (uint32_t i = 0; i < p.I; ++i) { const unsigned long long v = dbits(cs[i].abp.t_ab); if (v < bt) { bt = v; bs = SRC_ABP + i; } }
            for (uint32_t i = 0; i < p.I; ++i) { const unsigned long long v = dbits(cs[i].abd0.t_ab); if (v < bt) { bt = v; bs = SRC_ABD0 + i; } }
            for (uint32_t i = 0; i < p.I; ++i) { const unsigned long long v = dbits(cs[i].abd1.t_ab); if (v < bt) { bt = v; bs = SRC_ABD1 + i; } }
        }
        cl_t = bt; cl_s = bs; cl_valid = true;
    }

    __device__ __forceinline__ bool run()
    {
        const unsigned long long tend_bits = dbits(T_end);
        unsigned long long budget = p.event_budget;
        for (;;) {
            if (!cl_valid) class_candidates();
            // plain iteration ends, one after the other, while no other event comes first
            for (int k = 0; k < 4; ++k) {
                if (!nx_valid) peek();
                if (!(nx_t < cl_t) || nx_t > tend_bits || budget == 0 || err || !end_is_plain(nx_rec)) break;
                --budget;
                ++rounds;
                t = __longlong_as_double((long long)nx_t);
                plain_end();
            }
            if (!nx_valid) peek();
            if (err) return true;
            const bool server = nx_t < cl_t;            // a class event wins an exact tie (lower source id)
            const unsigned long long te = server ? nx_t : cl_t;
            if (te > tend_bits) return true;             // nothing left up to T_end (also when both are +inf)
            if (budget == 0) return false;
            --budget;
            ++rounds;
            t = __longlong_as_double((long long)te);
            if (server) {
                on_server();
            } else {
                const uint32_t src = cl_s;
                cl_valid = false;
                if (src >= SRC_ABD1) on_abandon_d(1, src - SRC_ABD1);
                else if (src >= SRC_ABD0) on_abandon_d(0, src - SRC_ABD0);
                else if (src >= SRC_ABP) on_abandon_p(src - SRC_ABP);
                else if (src >= SRC_ARRIVAL) on_arrival(src - SRC_ARRIVAL);
                else {
                    ++events;
                    const uint32_t M0 = M;
                    load_block(blk + 1);
                    if (M != M0) rebuild_trees();
                    drain_dirty = true; gate_dirty = true;
                }
            }
            if (err) return true;
            if (drain_dirty || gate_dirty || n_touch || touch_all) dispatch();
        }
    }
};

// Empty system at t = 0 for the one-thread-per-replication family: idle GPUs, empty calendar and trees, every slot of
// every GPU free, first arrival of every class scheduled, abandonment levels drawn.
__global__ void __launch_bounds__(32) qsim_lane_init_kernel(Params p)
{
    const uint32_t rep = blockIdx.x * blockDim.x + threadIdx.x;
    if (rep >= p.R) return;
    const LanePar &q = p.lane;
    LaneSim<LF_GENERIC> s(p, rep);
    s.bind();
    RepHeader &h = p.hdr[rep];
    s.cs = h.cs;               // set-up works on the records in global memory
    s.cg = NONE32;
    for (uint32_t o = 0; o < sizeof(RepHeader) / 8; ++o) reinterpret_cast<unsigned long long *>(&h)[o] = 0ull;
    for (uint32_t g = 0; g < p.N; ++g) {
        LaneSrv v;
        v.tnext = dinf(); v.it = 0; v.nfin = NONE32; v.pfjob = 0; v.pfrem = 0; v.pfcur = 0; v.ndec = 0; v.nact = 0; v.cnext = NONE16; v.ftop = NONE16;
        s.srv[g] = v;
        s.tarr[g] = 0.0;
        for (uint32_t j = 0; j < q.b8; ++j) s.sfin[(size_t)g * q.b8 + j] = NONE32;
        for (uint32_t j = 0; j < q.ssize; ++j) s.snode[(size_t)g * q.ssize + j] = ~0ull;
        for (uint32_t j = 0; j < p.B; ++j) s.sfree[(size_t)g * p.B + j] = (uint16_t)j;
    }
    for (uint32_t b = 0; b < q.nbk; ++b) s.chead[b] = (uint16_t)NONE16;
    for (uint32_t w = 0; w < (q.nbk >> 5); ++w) s.cbm[w] = 0u;      // nothing is inserted during set-up
    for (uint32_t w = 0; w < p.I * q.qw; ++w) s.pql[w] = 0u;
    s.err = 0;
    s.load_block(0);
    s.rebuild_trees();
    for (uint32_t i = 0; i < MAXI; ++i) {
        ClassState &c = h.cs[i];
        c.ta = dinf();
        AbClock *clk[3] = { &c.abp, &c.abd0, &c.abd1 };
        const uint32_t streams[3] = { STREAM_ABANDON_P, STREAM_ABANDON_D0, STREAM_ABANDON_D1 };
        for (int k = 0; k < 3; ++k) {
            uint32_t w0, w1, w2, w3;
            draw(p, rep, (streams[k] << 8) | i, 0, w0, w1, w2, w3);
            clk[k]->acc = 0.0; clk[k]->lvl = -qlog(u53(w0, w1)); clk[k]->t_last = 0.0; clk[k]->t_ab = dinf();
            clk[k]->m = 1;
        }
    }
    for (uint32_t i = 0; i < p.I; ++i) s.schedule_arrival(i, 0.0);
    h.err = s.err;
    if (p.hist_mem)
        for (uint32_t o = 0; o < p.I * 2 * NBIN; ++o) s.hist[o] = 0;
}

// Advance every replication to its new end time (or until the per-launch event budget runs out).
template <uint32_t LF>
__global__ void __launch_bounds__(32) qsim_lane_run_kernel(Params p)
{
    // A block is one warp; its first 1 << lsh lanes run a replication each.  With few replications the host picks
    // fewer lanes per warp: more warps run, and a warp waits for fewer lanes that took another branch.
    const uint32_t lpw = 1u << p.lane.lsh;
    const uint32_t rep = blockIdx.x * lpw + threadIdx.x;
    if (threadIdx.x >= lpw || rep >= p.R) return;
    RepHeader &h = p.hdr[rep];
    if (!p.advance && h.done) return;
    LaneSim<LF> s(p, rep);
    s.bind();
    // this lane's part of shared memory: class records (stride padded so that the lanes' 8-byte accesses fall into
    // different banks) and the calendar bitmap, word-interleaved over the lanes
    extern __shared__ __align__(16) uint32_t lane_sm[];
    const LanePar &lq = p.lane;
    s.cs = reinterpret_cast<ClassState *>(lane_sm + (size_t)threadIdx.x * lq.cs_stride);
    s.sbm = lane_sm + (size_t)lpw * lq.cs_stride + threadIdx.x;
    s.cg = NONE32;
    {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(h.cs);
        uint32_t *dst = reinterpret_cast<uint32_t *>(s.cs);
        for (uint32_t o = 0; o < p.I * (uint32_t)(sizeof(ClassState) / 4); ++o) dst[o] = src[o];
        for (uint32_t w = 0; w < (lq.nbk >> 5); ++w) s.bm(w) = s.cbm[w];
    }
    // the end time is one rounded product of the cumulative horizon: run(a); run(b) ends where run(a+b) ends
    double T_end = h.T_end;
    const unsigned long long H_total = h.H_total + (p.advance == 1 ? p.horizon_iters : 0ull);
    if (p.advance == 1) T_end = __dmul_rn((double)H_total, iter_time(p, 0, p.B, 0));
    if (p.advance == 2) T_end = p.T_abs;
    s.T_end = T_end;
    s.T_reset = h.T_reset;
    s.t = h.t_now;
    s.err = h.err;
    s.load_block(h.blk);
    s.dq_head0 = h.dq_head0; s.dq_head1 = h.dq_head1; s.dq_n0 = h.dq_n0; s.dq_n1 = h.dq_n1;
    s.events = h.events; s.rounds = h.rounds;
    s.it_mixed = h.iters_mixed[0]; s.it_solo = h.iters_solo[0]; s.busy_mixed = h.busy_mixed[0]; s.busy_solo = h.busy_solo[0];
    {
        const LanePar &q = p.lane;
        s.root_solo = s.tsolo[q.toff[q.tlev]]; s.root_mix = s.tmix[q.toff[q.tlev]]; s.root_pf = s.tpf[q.toff[q.tlev]];
    }
    s.nx_valid = false; s.cl_valid = false;
    s.n_touch = 0; s.touch_all = false; s.drain_dirty = true; s.gate_dirty = true;
    if (p.force_dispatch) s.rebuild_trees();     // the policy parameters were replaced: M may have changed
    const bool finished = s.err ? true : s.run();
    {
        uint32_t *dst = reinterpret_cast<uint32_t *>(h.cs);
        const uint32_t *src = reinterpret_cast<const uint32_t *>(s.cs);
        for (uint32_t o = 0; o < p.I * (uint32_t)(sizeof(ClassState) / 4); ++o) dst[o] = src[o];
        for (uint32_t w = 0; w < (lq.nbk >> 5); ++w) s.cbm[w] = s.bm(w);
    }
    h.T_end = T_end; h.H_total = H_total; h.blk = s.blk; h.t_now = s.t;
    h.dq_head0 = s.dq_head0; h.dq_head1 = s.dq_head1; h.dq_n0 = s.dq_n0; h.dq_n1 = s.dq_n1;
    h.events = s.events; h.rounds = s.rounds; h.err = s.err;
    h.iters_mixed[0] = s.it_mixed; h.iters_solo[0] = s.it_solo; h.busy_mixed[0] = s.busy_mixed; h.busy_solo[0] = s.busy_solo;
    h.done = finished ? 1u : 0u;
    if (!finished) atomicAdd(p.not_done, 1u);
}

}  // namespace qsimdev
