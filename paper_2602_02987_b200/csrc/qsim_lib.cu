// Host side of libqsim: the C ABI declared in include/qsim.h.
// Validates arguments, lays out the caller's workspace, launches the kernels of qsim_device.cuh and
// converts the device records into the public statistics structs.  No CPU simulation path exists here:
// without a CUDA device every entry point that needs one fails with QSIM_ECUDA.
#include "qsim.h"
#include "qsim_device.cuh"
#include "qsim_lane.cuh"

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using namespace qsimdev;

namespace {

thread_local std::string g_err;

int fail(int code, const std::string &msg)
{
    g_err = msg;
    return code;
}

#define CUDA_TRY(expr)                                                                         \
    do {                                                                                       \
        cudaError_t e_ = (expr);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return fail(QSIM_ECUDA, std::string(#expr) + ": " + cudaGetErrorString(e_));       \
    } while (0)

size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

struct TotalsRecBytes { char b[2048]; };      // room for the device totals record (checked where the record is defined)

struct Sections {
    size_t hdr, srv, fin, rec, pq, dq, hist, flag, red, tarr, total;
    // one-thread-per-replication family
    size_t l_srv, l_tarr, l_head, l_bm, l_tree, l_sfin, l_snode, l_srec, l_sfree, l_pql;
};

}  // namespace

struct qsim {
    qsim_config cfg{};
    qsim_class cls[QSIM_MAXI]{};
    double prices[2]{};
    Params par{};
    SmemLayout lay{};
    uint32_t init_smem = 0;       // shared memory of the set-up kernel's block (one warp, same per-GPU image)
    Sections sec{};
    BlockPar *d_blocks = nullptr;
    uint32_t *d_lengths = nullptr;
    double *d_inject_t = nullptr;
    uint32_t *d_inject_job = nullptr;
    uint32_t feat = 0;
    double T_end_abs = 0.0;       // end time reached by qsim_run_until calls
    bool targets_changed = false; // qsim_set_targets since the last launch
    uint32_t *h_flag = nullptr;   // pinned
    void *ws = nullptr;
    cudaStream_t stream = nullptr;
    bool bound = false;
    uint64_t launches = 0;
    uint32_t resident_blocks = 0; // blocks of run_fn that one device holds at a time (0 = not asked yet)
    uint32_t chunk_K = 1;         // chunks per replication of the launch in progress (see plan_chunks)
    uint64_t chunk_H = 0;         // and its horizon
    uint32_t tag_base = 0;        // hand-over stamps of this handle's launches start above every stamp in the workspace
    int device = 0;
    void (*run_fn)(qsimdev::Params) = nullptr;
    uint32_t nwarps = 1;          // warps per replication (block size / 32)
    void (*lane_fn)(qsimdev::Params) = nullptr;     // instance of the one-thread-per-replication run kernel
    bool allow_lane = true;       // the one-thread-per-replication family may run this handle
    double coef[6]{};
};

namespace {

Sections layout_sections(const qsim_config &c, uint32_t srv_bytes, bool tarr_global)
{
    Sections s{};
    size_t o = 0;
    const size_t R = c.R, NB = (size_t)c.N * c.B;
    s.hdr = o; o = align256(o + R * sizeof(RepHeader));
    s.srv = o; o = align256(o + R * (size_t)srv_bytes);
    s.fin = o; o = align256(o + R * NB * 4);
    s.rec = o; o = align256(o + R * NB * sizeof(SlotRec));
    s.pq = o; o = align256(o + R * (size_t)c.I * c.qcap * sizeof(QEntry));
    s.dq = o; o = align256(o + R * (size_t)2 * c.qcap * sizeof(QEntry));
    s.hist = o; if (c.hist) o = align256(o + R * (size_t)c.I * 2 * NBIN * 4);
    s.flag = o; o = align256(o + 256);
    s.red = o; o = align256(o + sizeof(TotalsRecBytes) + R * (size_t)(c.I * 7u + 3u) * 8);    // totals record + fp64 statistics per replication
    s.tarr = o; if (tarr_global) o = align256(o + R * (size_t)c.N * 12);      // arrival time (8 bytes) and job word (4) of the request in prefill
    s.total = o;
    return s;
}

Sections lane_sections(const qsim_config &c, const LanePar &q)
{
    Sections s{};
    size_t o = 0;
    const size_t R = c.R, N = c.N;
    s.hdr = o; o = align256(o + R * sizeof(RepHeader));
    s.l_srv = o; o = align256(o + R * N * sizeof(LaneSrv));
    s.l_tarr = o; o = align256(o + R * N * 8);
    s.l_head = o; o = align256(o + R * (size_t)q.nbk * 2);
    s.l_bm = o; o = align256(o + R * (size_t)(q.nbk / 32u) * 4);
    s.l_tree = o; o = align256(o + R * 3 * (size_t)q.tsize * 4);
    s.l_sfin = o; o = align256(o + R * N * (size_t)q.b8 * 4);
    s.l_snode = o; o = align256(o + R * N * (size_t)q.ssize * 8);
    s.l_srec = o; o = align256(o + R * N * (size_t)c.B * sizeof(SlotRec));
    s.l_sfree = o; o = align256(o + R * N * (size_t)c.B * 2);
    s.l_pql = o; o = align256(o + R * (size_t)c.I * q.qw * 4);
    s.pq = o; o = align256(o + R * (size_t)c.I * c.qcap * sizeof(QEntry));
    s.dq = o; o = align256(o + R * (size_t)2 * c.qcap * sizeof(QEntry));
    s.hist = o; if (c.hist) o = align256(o + R * (size_t)c.I * 2 * NBIN * 4);
    s.flag = o; o = align256(o + 256);
    s.red = o; o = align256(o + sizeof(TotalsRecBytes) + R * (size_t)(c.I * 7u + 3u) * 8);    // totals record + fp64 statistics per replication
    s.total = o;
    return s;
}

// 8-ary tree over n leaves: number of internal levels, offset of every level (level 0 = leaves) and total entries;
// every level is padded to a multiple of eight entries.
void tree_shape(uint32_t n, uint32_t &lev, uint32_t *off, uint32_t &size)
{
    uint32_t m = (n + 7u) & ~7u, o = 0;
    lev = 0;
    off[0] = 0;
    for (;;) {
        o += m;
        const uint32_t parents = (m + 7u) / 8u;
        ++lev;
        off[lev] = o;
        if (parents == 1) { size = o + 8u; return; }
        m = (parents + 7u) & ~7u;
    }
}

// Which configurations the one-thread-per-replication family simulates: every gate, the solo-first and the SLI-aware
// router with least-loaded placement, abandonment, blocks, histograms; no KV slope, no trace replay.
bool lane_supports(const qsim_config &c, const double *coef)
{
    return (c.router == QSIM_ROUTER_SOLO_FIRST || c.router == QSIM_ROUTER_SLI) && c.placement == QSIM_PLACE_LEAST_LOADED &&
           coef[5] == 0.0 && c.N <= 4096 && c.B <= 4096;
}

// Shapes of the family's structures (no pointers yet)
void lane_shapes(const qsim_config &c, const double *coef, LanePar &q)
{
    std::memset(&q, 0, sizeof q);
    q.on = 1;
    uint32_t nbk = 64;
    while (nbk < 4u * c.N) nbk <<= 1;
    q.nbk = nbk;
    // no iteration lasts longer than tau_max, so with (nbk - 2) buckets per 1.01 tau_max every pending end lies less
    // than one revolution of the calendar ahead of the current time
    const double tau_mix = coef[0] + coef[1] * (double)c.C + coef[2] * (double)c.B, tau_solo = coef[3] + coef[4] * (double)c.B;
    const double tau_max = tau_mix > tau_solo ? tau_mix : tau_solo;
    q.inv_w = (double)(nbk - 2u) / (1.01 * tau_max);
    tree_shape(c.N, q.tlev, q.toff, q.tsize);
    q.b8 = (c.B + 7u) & ~7u;
    uint32_t off[6], size = 0;
    tree_shape(c.B, q.slev, off, size);
    for (uint32_t l = 0; l < q.slev; ++l) q.soff[l] = off[l + 1] - off[1];      // internal levels only: the leaves are a separate array
    q.ssize = size - off[1];
    q.qw = ((c.qcap + 127u) / 128u) * 4u;
    // replications per warp: 32 when there are enough of them for 512 warps, else 16 or 8 (measured at 1024 and 4096 GPUs
    // with 4096 and 8192 replications: +12 % and +10 % over 32; 4 per warp is slower again); QSIM_LANE_LSH overrides (2..5)
    q.lsh = 5;
    while (q.lsh > 3 && (c.R >> q.lsh) < 512u) --q.lsh;
    if (const char *e = std::getenv("QSIM_LANE_LSH")) {
        const int v = std::atoi(e);
        if (v >= 2 && v <= 5) q.lsh = (uint32_t)v;
    }
    // shared memory of a block: per lane the class records, at a stride whose half is odd (the lanes' 8-byte
    // accesses then fall into different banks), and one bit per calendar bucket
    uint32_t stride = c.I * (uint32_t)(sizeof(ClassState) / 4);
    if (((stride / 2u) & 1u) == 0) stride += 2u;
    q.cs_stride = stride;
    q.smem_bytes = (1u << q.lsh) * (stride * 4u + q.nbk / 8u);
}

int validate(const qsim_config *cfg, const qsim_class *classes, const double *rates, const uint32_t *lengths,
             const double *prices, const double *coef, const qsim_targets *tg)
{
    if (!cfg || !classes || !rates || !prices || !coef || !tg) return fail(QSIM_EINVAL, "null argument");
    if (cfg->size != sizeof(qsim_config)) return fail(QSIM_EINVAL, "qsim_config.size does not match this library");
    if (cfg->I < 1 || cfg->I > QSIM_MAXI) return fail(QSIM_EINVAL, "I must be in 1..8");
    if (cfg->N < 1 || cfg->N > 4096) return fail(QSIM_EINVAL, "N must be in 1..4096");
    if (cfg->R < 1) return fail(QSIM_EINVAL, "R must be >= 1");
    if (cfg->B < 1 || cfg->B > 4096) return fail(QSIM_EINVAL, "B must be in 1..4096");
    if (cfg->C < 1 || cfg->C > 65535) return fail(QSIM_EINVAL, "C must be in 1..65535");
    if (cfg->nblk < 1) return fail(QSIM_EINVAL, "nblk must be >= 1");
    if (cfg->qcap < 1 || cfg->qcap > (1u << 24)) return fail(QSIM_EINVAL, "qcap must be in 1..2^24");
    if (cfg->gate > 2 || cfg->router > 3 || cfg->placement > 1 || cfg->pricing > 1 || cfg->length_mode > 1 || cfg->hist > 1)
        return fail(QSIM_EINVAL, "enum out of range");
    if (cfg->nblk > 1 && !(cfg->block_len > 0.0 && std::isfinite(cfg->block_len)))
        return fail(QSIM_EINVAL, "block_len must be positive when nblk > 1");
    if (cfg->length_mode == QSIM_LENGTH_TABLE && !lengths) return fail(QSIM_EINVAL, "length tables missing");
    for (uint32_t i = 0; i < cfg->I; ++i) {
        if (classes[i].P < 1 || classes[i].P > QSIM_LMAX || classes[i].D < 1 || classes[i].D > QSIM_LMAX)
            return fail(QSIM_EINVAL, "class lengths must be in 1..8192");
        if (!(classes[i].theta >= 0.0) || !std::isfinite(classes[i].theta)) return fail(QSIM_EINVAL, "theta must be >= 0");
    }
    for (size_t k = 0; k < (size_t)cfg->nblk * cfg->I; ++k)
        if (!(rates[k] >= 0.0) || !std::isfinite(rates[k])) return fail(QSIM_EINVAL, "rates must be finite and >= 0");
    for (int k = 0; k < 6; ++k)
        if (!std::isfinite(coef[k]) || coef[k] < 0.0) return fail(QSIM_EINVAL, "iteration-time coefficients must be finite and >= 0");
    if (!(coef[0] > 0.0) || !(coef[3] > 0.0)) return fail(QSIM_EINVAL, "alpha_m and alpha_s must be positive");
    if (!std::isfinite(prices[0]) || !std::isfinite(prices[1])) return fail(QSIM_EINVAL, "prices must be finite");
    for (uint32_t b = 0; b < cfg->nblk; ++b) {
        if (tg[b].M > cfg->N) return fail(QSIM_EINVAL, "M must be <= N");
        for (uint32_t i = 0; i < cfg->I; ++i) {
            if (!std::isfinite(tg[b].xstar[i]) || tg[b].xstar[i] < 0.0 || !std::isfinite(tg[b].n_xstar[i]) ||
                !std::isfinite(tg[b].n_qpstar[i]) || !(tg[b].p_solo[i] >= 0.0 && tg[b].p_solo[i] <= 1.0) ||
                !(tg[b].w_solo[i] >= 0.0) || !std::isfinite(tg[b].w_solo[i]) || !(tg[b].w_mix[i] >= 0.0) || !std::isfinite(tg[b].w_mix[i]))
                return fail(QSIM_EINVAL, "LP targets out of range");
        }
    }
    if (lengths && cfg->length_mode == QSIM_LENGTH_TABLE)
        for (uint32_t t = 0; t < cfg->I * 2; ++t) {
            const uint32_t *thr = lengths + (size_t)t * QSIM_LMAX;
            for (uint32_t j = 1; j < QSIM_LMAX - 1; ++j)
                if (thr[j] < thr[j - 1]) return fail(QSIM_EINVAL, "length thresholds must be non-decreasing");
        }
    return QSIM_OK;
}

// Threshold tables as the kernels read them: the caller's [I][2][LMAX] words followed by a coarse index per table
// (entry b = number of thresholds below b 2^24, b = 0..256), which narrows the binary search of a draw to one bucket.
size_t table_bytes(uint32_t I) { return (size_t)I * 2 * QSIM_LMAX * 4 + (size_t)I * 2 * LIDX * 2; }

std::vector<uint32_t> tables_with_index(const uint32_t *lengths, uint32_t I)
{
    std::vector<uint32_t> buf(table_bytes(I) / 4, 0u);
    std::memcpy(buf.data(), lengths, (size_t)I * 2 * QSIM_LMAX * 4);
    uint16_t *idx = reinterpret_cast<uint16_t *>(buf.data() + (size_t)I * 2 * QSIM_LMAX);
    for (uint32_t t = 0; t < I * 2; ++t) {
        const uint32_t *thr = lengths + (size_t)t * QSIM_LMAX;
        uint32_t j = 0;
        for (uint32_t b = 0; b <= 256; ++b) {
            const uint64_t bound = (uint64_t)b << 24;
            while (j < QSIM_LMAX - 1 && thr[j] < bound) ++j;
            idx[(size_t)t * LIDX + b] = (uint16_t)j;
        }
    }
    return buf;
}

// Instances of the run kernel: (GPUs per lane, feature set).  A problem runs on the smallest instance that
// contains its features; the fully generic instance takes everything else.
using RunKernel = void (*)(Params);
struct RunVariant { int spl; uint32_t feat; RunKernel fn; };

template <int SPL>
void add_variants(std::vector<RunVariant> &v)
{
    v.push_back({SPL, F_SLOTS, qsim_run_kernel<SPL, F_SLOTS>});
    v.push_back({SPL, F_SLOTS | F_OCC, qsim_run_kernel<SPL, F_SLOTS | F_OCC>});
    v.push_back({SPL, F_SLOTS | F_OCC | F_ABANDON, qsim_run_kernel<SPL, F_SLOTS | F_OCC | F_ABANDON>});
    v.push_back({SPL, F_SLOTS | F_OCC | F_ABANDON | F_RANDOM, qsim_run_kernel<SPL, F_SLOTS | F_OCC | F_ABANDON | F_RANDOM>});
    // occupancy gate with abandonment when the finish stamps do not fit on chip (large B), and the SLI-aware router with
    // histograms in both slot modes
    v.push_back({SPL, F_OCC | F_ABANDON, qsim_run_kernel<SPL, F_OCC | F_ABANDON>});
    v.push_back({SPL, F_OCC | F_ABANDON | F_SLI | F_HIST, qsim_run_kernel<SPL, F_OCC | F_ABANDON | F_SLI | F_HIST>});
    v.push_back({SPL, F_SLOTS | F_OCC | F_ABANDON | F_SLI | F_HIST, qsim_run_kernel<SPL, F_SLOTS | F_OCC | F_ABANDON | F_SLI | F_HIST>});
    v.push_back({SPL, F_GENERIC, qsim_run_kernel<SPL, F_GENERIC>});
}

const std::vector<RunVariant> &run_variants()
{
    static const std::vector<RunVariant> table = [] {
        std::vector<RunVariant> v;
        add_variants<1>(v);
        add_variants<2>(v);
        add_variants<4>(v);
        // one warp, run-time row count (129..511 GPUs)
        v.push_back({0, F_OCC | F_ABANDON, qsim_run_kernel<0, F_OCC | F_ABANDON>});
        v.push_back({0, F_OCC | F_ABANDON | F_SLI | F_HIST, qsim_run_kernel<0, F_OCC | F_ABANDON | F_SLI | F_HIST>});
        v.push_back({0, F_GENERIC, qsim_run_kernel<0, F_GENERIC>});
        // several warps per replication (large clusters): instances for the occupancy gate with abandonment under
        // the solo-first and (with histograms) the SLI-aware router, the priority gate with blocks and histograms, and the generic one
        v.push_back({-1, F_MW | F_OCC | F_ABANDON, qsim_run_kernel<0, F_MW | F_OCC | F_ABANDON>});
        v.push_back({-1, F_MW | F_OCC | F_ABANDON | F_SLI | F_HIST, qsim_run_kernel<0, F_MW | F_OCC | F_ABANDON | F_SLI | F_HIST>});
        v.push_back({-1, F_MW | F_ABANDON | F_BLOCKS | F_HIST, qsim_run_kernel<0, F_MW | F_ABANDON | F_BLOCKS | F_HIST>});
        v.push_back({-1, F_GENERIC | F_MW, qsim_run_kernel<0, F_GENERIC | F_MW>});
        return v;
    }();
    return table;
}

uint32_t features_of(const qsim_config &c, const qsim_class *cls, const double *coef)
{
    uint32_t f = 0;
    for (uint32_t i = 0; i < c.I; ++i)
        if (cls[i].theta > 0.0) f |= F_ABANDON;
    if (c.router == QSIM_ROUTER_SLI) f |= F_SLI;
    if (c.router == QSIM_ROUTER_SLI_GENERAL) f |= F_SLI | F_SLIG;
    if (c.router == QSIM_ROUTER_IMMEDIATE) f |= F_IMM;
    if (coef[5] != 0.0) f |= F_KAPPA;
    if (c.hist) f |= F_HIST;
    if (c.nblk > 1) f |= F_BLOCKS;
    if (c.placement == QSIM_PLACE_RANDOM) f |= F_RANDOM;
    if (c.gate == QSIM_GATE_OCCUPANCY) f |= F_OCC;
    if (c.gate == QSIM_GATE_FCFS) f |= F_FCFS;
    return f;
}

// Large clusters: per-replication shared memory allows only a few blocks per SM, so each replication gets
// several warps (master + helpers) that share the per-GPU scans.  QSIM_WARPS overrides the choice (1 = off).
void choose_multiwarp(uint32_t N, uint32_t feat, Params &p, RunKernel &fn, uint32_t &nwarps)
{
    const uint32_t rows = (N + 31u) / 32u;
    uint32_t W = rows >= 128 ? 16u : (rows >= 64 ? 4u : (rows >= 32 ? 2u : 1u));     // best of sweeps over 1, 2, 4, 8, 16 warps at 512, 768, 1024, 2048, 4096 GPUs
    if (const char *e = std::getenv("QSIM_WARPS")) {
        const int v = std::atoi(e);
        if (v >= 1 && v <= MW_MAX) W = (uint32_t)v;
    }
    if (W <= 1 || rows < 2) return;
    const char *force = std::getenv("QSIM_KERNEL");
    const bool generic_only = force && std::strcmp(force, "generic") == 0;
    // mode bits must match exactly, capability bits may be present unused (as in pick_run_kernel)
    constexpr uint32_t MODES = F_SLI | F_SLIG | F_IMM | F_RANDOM | F_OCC | F_FCFS | F_HIST;
    const RunVariant *best = nullptr;
    int best_bits = 99;
    for (const RunVariant &v : run_variants()) {
        if (v.spl >= 0) continue;
        if (v.feat & F_GENERIC) { if (!best) best = &v; continue; }
        if (generic_only || (feat & MODES) != (v.feat & MODES) || (feat & ~(v.feat | F_SLOTS)) != 0) continue;
        const int extra = __builtin_popcount(v.feat & ~feat & ~F_MW);
        if (extra < best_bits) { best = &v; best_bits = extra; }
    }
    fn = best->fn;
    nwarps = W;
    p.Npad = rows * 32u;
    p.slots_smem = 0;       // helpers retire through the global slot lists
}

RunVariant pick_run_kernel(uint32_t N, uint32_t feat)
{
    const int rows = (int)((N + 31u) / 32u);
    const RunVariant *generic = nullptr, *best = nullptr;
    // QSIM_KERNEL=generic forces the run-time-configured instance (for cross-checking the specialised ones)
    const char *force = std::getenv("QSIM_KERNEL");
    if (force && std::strcmp(force, "generic") == 0) feat = ~0u;
    int best_bits = 99;
    for (const RunVariant &v : run_variants()) {
        if (v.spl < 0) continue;                            // the multi-warp instance is chosen by the caller
        if (v.spl != 0 && v.spl < rows) continue;          // too few GPUs per lane
        if (v.spl == 0 && (v.feat & F_GENERIC)) { generic = &v; continue; }
        // smallest row count that fits (0 = run-time row count, beyond four rows); among those the feature set with
        // the fewest extras
        int spl_fit = rows <= 1 ? 1 : (rows <= 2 ? 2 : (rows <= 4 ? 4 : 0));
        if (v.spl != spl_fit) continue;
        if (v.feat & F_GENERIC) { if (!best) { best = &v; best_bits = 98; } continue; }
        // mode bits (router, placement, gate, histograms) select code and must match exactly; capability bits
        // (abandonment, KV slope, blocks) may be present without being used
        constexpr uint32_t MODES = F_SLI | F_SLIG | F_IMM | F_RANDOM | F_OCC | F_FCFS | F_HIST | F_SLOTS;
        if (feat == ~0u || (feat & MODES) != (v.feat & MODES) || (feat & ~v.feat) != 0) continue;
        const int extra = __builtin_popcount(v.feat & ~feat);
        if (extra < best_bits) { best = &v; best_bits = extra; }
    }
    return best ? *best : *generic;
}

// Everything of a handle that needs no device memory: kernel parameters, kernel instance, block shape,
// shared-memory and workspace layouts.
int configure(qsim &h, const qsim_config &cfg, const qsim_class *classes, const double *prices, const double *coef)
{
    h.cfg = cfg;
    if (classes != h.cls) std::memcpy(h.cls, classes, cfg.I * sizeof(qsim_class));
    h.prices[0] = prices[0];
    h.prices[1] = prices[1];
    Params &p = h.par;
    p.I = cfg.I; p.N = cfg.N; p.Npad = (cfg.N + 31u) & ~31u; p.R = cfg.R; p.B = cfg.B; p.C = cfg.C;
    p.nblk = cfg.nblk; p.gate = cfg.gate; p.router = cfg.router; p.placement = cfg.placement;
    p.length_mode = cfg.length_mode; p.qcap = cfg.qcap; p.hist = cfg.hist;
    p.seed = cfg.seed; p.rep_offset = cfg.rep_offset; p.block_len = cfg.block_len;
    p.event_budget = 1ull << 28;
    p.any_theta = 0;
    for (int k = 0; k < 6; ++k) p.coef[k] = coef[k];
    for (uint32_t i = 0; i < cfg.I; ++i) {
        p.cls[i].theta = classes[i].theta; p.cls[i].P = classes[i].P; p.cls[i].D = classes[i].D;
        p.cls[i].prio = classes[i].prio_rank; p.cls[i].pad = 0;
        if (classes[i].theta > 0.0) p.any_theta = 1;
    }
    const bool kappa = coef[5] != 0.0;
    const uint32_t feat = features_of(cfg, classes, coef);
    RunVariant v = pick_run_kernel(cfg.N, feat);
    // the per-GPU arrays are padded to the unrolled row count of the chosen instance
    if (v.spl > 0) p.Npad = (uint32_t)v.spl * 32u;
    // finish stamps + occupancy bits go to shared memory when the whole block state stays small
    p.slots_smem = smem_layout(p.Npad, p.B, 1, 1, kappa, p.Npad > 128u, cfg.I).total <= 40u * 1024u ? 1u : 0u;
    if (p.slots_smem) v = pick_run_kernel(cfg.N, feat | F_SLOTS);
    h.run_fn = v.fn;
    h.nwarps = 1;
    choose_multiwarp(cfg.N, feat, p, h.run_fn, h.nwarps);
    // beyond four rows of GPUs shared memory limits the resident replications: the arrival times and the job words of
    // the requests in prefill (read once per finished prefill) move to global memory
    p.tarr_global = (p.Npad > 128u) ? 1u : 0u;
    h.lay = smem_layout(p.Npad, p.B, p.slots_smem, h.nwarps, kappa, p.tarr_global != 0, cfg.I);
    h.init_smem = smem_layout(p.Npad, p.B, p.slots_smem, 1, kappa, p.tarr_global != 0, cfg.I).total;
    p.srv_bytes = h.lay.srv_bytes;
    if (h.lay.total > 227u * 1024u - 64u)       // a few bytes of the block are the kernel's own
        return fail(QSIM_EINVAL, "N too large: per-replication GPU state does not fit shared memory");
    h.sec = layout_sections(cfg, p.srv_bytes, p.tarr_global != 0);
    for (int k = 0; k < 6; ++k) h.coef[k] = coef[k];
    // Kernel family.  A replication advances at about the same rate on one thread whatever its cluster size, while the
    // warp-per-replication kernels slow down in proportion to the cluster (few replications fit on an SM and their
    // master warp searches all rows).  Measured on a B200: one thread per replication wins from 2048 GPUs when R x N
    // exceeds about 7 million (N = 2048, R = 4096: 2.26e8 against 2.18e8 it/s; N = 4096, R = 4096: 2.1e8 against 5.3e7),
    // and not below (N = 1024: 3.35e8 against 3.47e8 at R = 8192, 3.15e8 against 3.53e8 at R = 16384; N = 512,
    // R = 16384: 3.5e8 against 7e8).  QSIM_FAMILY=lane / warp overrides.
    std::memset(&p.lane, 0, sizeof p.lane);
    bool lane = h.allow_lane && lane_supports(cfg, coef) && cfg.N >= 2048u && (unsigned long long)cfg.R * cfg.N >= 7000000ull;
    if (const char *e = std::getenv("QSIM_FAMILY")) {
        if (std::strcmp(e, "lane") == 0) lane = h.allow_lane && lane_supports(cfg, coef);
        else if (std::strcmp(e, "warp") == 0) lane = false;
    }
    if (lane) {
        // the smallest instance that contains the configuration's features
        const bool ab = p.any_theta != 0, sli = cfg.router == QSIM_ROUTER_SLI, hist = cfg.hist != 0, blk = cfg.nblk > 1;
        const char *force = std::getenv("QSIM_KERNEL");
        if (force && std::strcmp(force, "generic") == 0) h.lane_fn = qsim_lane_run_kernel<LF_GENERIC>;
        else if (!sli && !hist && !blk) h.lane_fn = ab ? qsim_lane_run_kernel<LF_ABANDON> : qsim_lane_run_kernel<0u>;
        else if (sli && hist && !blk) h.lane_fn = qsim_lane_run_kernel<LF_ABANDON | LF_SLI | LF_HIST>;
        else if (!sli && blk && hist) h.lane_fn = qsim_lane_run_kernel<LF_ABANDON | LF_BLOCKS | LF_HIST>;
        else h.lane_fn = qsim_lane_run_kernel<LF_GENERIC>;       // (abandonment code with theta = 0 is inert, so it may be compiled in)
        lane_shapes(cfg, coef, p.lane);
        if (p.lane.smem_bytes > 227u * 1024u) return fail(QSIM_EINVAL, "class records and calendar do not fit shared memory");
        h.sec = lane_sections(cfg, p.lane);
        h.nwarps = 0;
    }
    return QSIM_OK;
}

// Dynamic shared memory above 48 KB must be allowed per kernel.  The limit belongs to the kernel, not to a handle, and
// handles of different sizes share kernels: it is raised to the most the device allows and never lowered.
cudaError_t allow_large_smem(const void *fn)
{
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    cudaFuncAttributes fa{};
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, fn);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);   // the kernel's static part counts too
    return e;
}

void fill_blocks(BlockPar *blocks, const qsim_config &cfg, const double *rates, const qsim_targets *tg)
{
    for (uint32_t b = 0; b < cfg.nblk; ++b) {
        BlockPar &bp = blocks[b];
        std::memset(&bp, 0, sizeof bp);
        bp.M = tg[b].M;
        for (uint32_t i = 0; i < cfg.I; ++i) {
            bp.xstar[i] = tg[b].xstar[i]; bp.nx[i] = tg[b].n_xstar[i]; bp.nq[i] = tg[b].n_qpstar[i];
            bp.ps[i] = tg[b].p_solo[i]; bp.ws[i] = tg[b].w_solo[i]; bp.wm[i] = tg[b].w_mix[i]; bp.rate[i] = rates[(size_t)b * cfg.I + i];
        }
    }
}

// When the replications outnumber the blocks the device holds at a time, but not by much, a launch of one block per
// replication ends with a nearly empty last wave.  Such a launch is run as K chunks of the horizon per replication by one
// block per resident slot (qsim_run_kernel), with K the smallest count that fills the last wave to 97 % (chunks of at
// least 32 iterations of horizon, at most 64 chunks).  QSIM_CHUNKS overrides the choice (1 = off).
uint32_t plan_chunks(qsim *h, uint64_t horizon)
{
    if (h->par.lane.on) return 1;
    if (h->resident_blocks == 0) {
        int per_sm = 0, sms = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reinterpret_cast<const void *>(h->run_fn), (int)(32 * h->nwarps), h->lay.total) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess || per_sm < 1 || sms < 1) {
            cudaGetLastError();
            return 1;
        }
        h->resident_blocks = (uint32_t)per_sm * (uint32_t)sms;
    }
    const uint64_t R = h->cfg.R, G = h->resident_blocks, max_K = std::min<uint64_t>(64, horizon / 32);
    if (const char *e = std::getenv("QSIM_CHUNKS")) {
        const long v = std::atol(e);
        return (uint32_t)std::max<long>(1, std::min<long>(v, (long)std::max<uint64_t>(max_K, 1)));
    }
    if (R <= G || R * 64 >= (1ull << 32)) return 1;
    auto fill = [&](uint64_t K) { return (double)(K * R) / (double)(((K * R + G - 1) / G) * G); };
    if (fill(1) >= 0.95) return 1;
    uint64_t best = 1;
    for (uint64_t K = 2; K <= max_K; ++K) {
        if (fill(K) > fill(best) + 1e-9) best = K;
        if (fill(best) >= 0.97) break;
    }
    return (uint32_t)best;
}

int launch_run(qsim *h, uint32_t advance, uint64_t horizon, double T_abs = 0.0)
{
    Params p = h->par;
    p.advance = advance;
    p.horizon_iters = horizon;
    p.T_abs = T_abs;
    p.force_dispatch = h->targets_changed ? 1u : 0u;
    h->targets_changed = false;
    if (advance == 1) { h->chunk_K = plan_chunks(h, horizon); h->chunk_H = horizon; }
    else if (advance == 2) h->chunk_K = 1;
    // a launch that continues a chunked one (advance 0) keeps its chunks: every replication goes on where it stopped
    p.nchunk = h->chunk_K;
    if (p.nchunk > 1) p.horizon_iters = h->chunk_H;
    h->launches++;
    p.launch_tag = (h->tag_base + (uint32_t)h->launches) << 8;
    CUDA_TRY(cudaMemsetAsync(p.not_done, 0, 12, h->stream));
    if (p.lane.on) h->lane_fn<<<(h->cfg.R + (1u << p.lane.lsh) - 1u) >> p.lane.lsh, 32, p.lane.smem_bytes, h->stream>>>(p);
    else h->run_fn<<<p.nchunk > 1 ? h->resident_blocks : h->cfg.R, 32 * h->nwarps, h->lay.total, h->stream>>>(p);
    CUDA_TRY(cudaGetLastError());
    CUDA_TRY(cudaMemcpyAsync(h->h_flag, p.not_done, 12, cudaMemcpyDeviceToHost, h->stream));
    return QSIM_OK;
}

// After the stream has been synchronised: did every replication reach its end time (1), are more launches needed (0), or
// did a block give up waiting for a chunk (error)?
int launch_outcome(const qsim *h, bool &finished)
{
    if (h->h_flag[2] != 0) return fail(QSIM_ECUDA, "a block gave up waiting for the previous chunk of its replication; the state is not usable");
    finished = h->h_flag[0] == 0;
    return QSIM_OK;
}

}  // namespace

namespace {

// Statistics of one replication from its device record.  The same function runs on the host (qsim_stats with per-replication
// output) and on the device (totals only): every operation is one rounded IEEE double operation on either side.
__host__ __device__ inline void rep_stats_of(const RepHeader &H, uint32_t I, qsim_rep_stats &st)
{
    const double T = H.T_end;
    st.T_elapsed = T - H.T_reset;
    st.iters_mixed = 0; st.iters_solo = 0; st.busy_mixed = 0.0; st.busy_solo = 0.0;
    for (int l = 0; l < 32; ++l) {
        st.iters_mixed += H.iters_mixed[l];
        st.iters_solo += H.iters_solo[l];
        st.busy_mixed = st.busy_mixed + H.busy_mixed[l];
        st.busy_solo = st.busy_solo + H.busy_solo[l];
    }
    st.events = H.events + st.iters_mixed + st.iters_solo;   // H.events counts block switches; class events are added below
    for (uint32_t i = 0; i < I; ++i) {
        const ClassState &c = H.cs[i];
        qsim_class_stats &o = st.cls[i];
        o.arrivals = c.arrivals; o.admitted = c.admitted; o.prefill_done = c.prefill_done;
        o.placed_mixed = c.placed_mixed; o.placed_solo = c.placed_solo; o.done_mixed = c.done_mixed;
        o.done_solo = c.done_solo; o.abandoned_p = c.abandoned_p; o.abandoned_d = c.abandoned_d;
        o.overflow = c.overflow; o.overflow_d = c.overflow_d; o.tokens_in_prefilled = c.tok_in_pf;
        o.tokens_in_completed = c.tok_in_done; o.tokens_out_completed = c.tok_out_done;
        const uint32_t Qd = c.Qd0 + c.Qd1;
        o.Qp = c.pq_n; o.X = c.X; o.Qd = Qd; o.Ym = c.Ym; o.Ys = c.Ys; o.reserved = 0;
        // integrals are reported up to the end of the run without touching the stored state
        o.area_Qp = c.aQp.area + (double)c.pq_n * (T - c.aQp.t_last);
        o.area_X = c.aX.area + (double)c.X * (T - c.aX.t_last);
        o.area_Qd = c.aQd.area + (double)Qd * (T - c.aQd.t_last);
        o.area_Ym = (c.sYm_out - c.sYm_in) + (double)c.Ym * (T - H.T_reset);
        o.area_Ys = (c.sYs_out - c.sYs_in) + (double)c.Ys * (T - H.T_reset);
        o.sum_ttft = c.sum_ttft; o.sum_tpot = c.sum_tpot;
        st.events += c.arrivals + c.abandoned_p + c.abandoned_d;
    }
}

// One more replication into the totals (replications are added in index order, so the fp64 totals are reproducible)
inline void add_rep_stats(qsim_rep_stats &tot, const qsim_rep_stats &st, uint32_t I)
{
    tot.iters_mixed += st.iters_mixed; tot.iters_solo += st.iters_solo; tot.events += st.events;
    tot.busy_mixed += st.busy_mixed; tot.busy_solo += st.busy_solo; tot.T_elapsed += st.T_elapsed;
    for (uint32_t i = 0; i < I; ++i) {
        const qsim_class_stats &a = st.cls[i];
        qsim_class_stats &b = tot.cls[i];
        b.arrivals += a.arrivals; b.admitted += a.admitted; b.prefill_done += a.prefill_done;
        b.placed_mixed += a.placed_mixed; b.placed_solo += a.placed_solo; b.done_mixed += a.done_mixed;
        b.done_solo += a.done_solo; b.abandoned_p += a.abandoned_p; b.abandoned_d += a.abandoned_d;
        b.overflow += a.overflow; b.overflow_d += a.overflow_d; b.tokens_in_prefilled += a.tokens_in_prefilled;
        b.tokens_in_completed += a.tokens_in_completed; b.tokens_out_completed += a.tokens_out_completed;
        b.Qp += a.Qp; b.X += a.X; b.Qd += a.Qd; b.Ym += a.Ym; b.Ys += a.Ys;
        b.area_Qp += a.area_Qp; b.area_X += a.area_X; b.area_Qd += a.area_Qd; b.area_Ym += a.area_Ym;
        b.area_Ys += a.area_Ys; b.sum_ttft += a.sum_ttft; b.sum_tpot += a.sum_tpot;
    }
}

// Totals on the device (a11, statistics reduction).  Integer counters are summed with atomic additions (exact in any
// order); the floating-point statistics of every replication go to a compact array and one thread per statistic adds
// them in replication order, which is the order the host uses: the totals are bit-identical to the host's.
constexpr uint32_t NF_CLASS = 7, NF_REP = 3;      // fp64 statistics per class and per replication
struct TotalsRec { qsim_rep_stats tot; uint32_t err_rep, err_code; };
static_assert(sizeof(TotalsRec) <= sizeof(TotalsRecBytes), "room for the totals record in the workspace");

__global__ void qsim_totals_gather_kernel(const RepHeader *hdr, uint32_t R, uint32_t I, double *F, TotalsRec *out)
{
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= R) return;
    const RepHeader &H = hdr[r];
    if (H.err) { if (atomicCAS(&out->err_code, 0u, H.err) == 0u) out->err_rep = r; return; }
    qsim_rep_stats st;
    rep_stats_of(H, I, st);
    const uint32_t nf = I * NF_CLASS + NF_REP;
    double *f = F + (size_t)r * nf;
    qsim_rep_stats &t = out->tot;
    typedef unsigned long long u64;
    atomicAdd((u64 *)&t.iters_mixed, (u64)st.iters_mixed); atomicAdd((u64 *)&t.iters_solo, (u64)st.iters_solo);
    atomicAdd((u64 *)&t.events, (u64)st.events);
    for (uint32_t i = 0; i < I; ++i) {
        const qsim_class_stats &a = st.cls[i];
        qsim_class_stats &b = t.cls[i];
        const uint64_t *src = &a.arrivals;
        uint64_t *dst = &b.arrivals;
        for (int k = 0; k < 14; ++k) atomicAdd((u64 *)(dst + k), (u64)src[k]);      // the fourteen 64-bit counters are contiguous
        atomicAdd(&b.Qp, a.Qp); atomicAdd(&b.X, a.X); atomicAdd(&b.Qd, a.Qd); atomicAdd(&b.Ym, a.Ym); atomicAdd(&b.Ys, a.Ys);
        double *fc = f + i * NF_CLASS;
        fc[0] = a.area_Qp; fc[1] = a.area_X; fc[2] = a.area_Qd; fc[3] = a.area_Ym; fc[4] = a.area_Ys; fc[5] = a.sum_ttft; fc[6] = a.sum_tpot;
    }
    f[I * NF_CLASS + 0] = st.busy_mixed; f[I * NF_CLASS + 1] = st.busy_solo; f[I * NF_CLASS + 2] = st.T_elapsed;
}

__global__ void qsim_totals_sum_kernel(uint32_t R, uint32_t I, const double *F, TotalsRec *out)
{
    const uint32_t nf = I * NF_CLASS + NF_REP, k = threadIdx.x;
    if (k >= nf || out->err_code) return;
    double acc = 0.0;
    for (uint32_t r = 0; r < R; ++r) acc = acc + F[(size_t)r * nf + k];
    qsim_rep_stats &t = out->tot;
    if (k < I * NF_CLASS) {
        qsim_class_stats &b = t.cls[k / NF_CLASS];
        double *dst[NF_CLASS] = { &b.area_Qp, &b.area_X, &b.area_Qd, &b.area_Ym, &b.area_Ys, &b.sum_ttft, &b.sum_tpot };
        *dst[k % NF_CLASS] = acc;
    } else if (k == I * NF_CLASS) t.busy_mixed = acc;
    else if (k == I * NF_CLASS + 1) t.busy_solo = acc;
    else t.T_elapsed = acc;
}

}  // namespace

extern "C" {

const char *qsim_last_error(void) { return g_err.c_str(); }

int qsim_create(qsim_t **out, const qsim_config *cfg, const qsim_class *classes, const double *rates,
                const uint32_t *lengths, const double *prices, const double *coef, const qsim_targets *tg)
{
    if (!out) return fail(QSIM_EINVAL, "null out pointer");
    *out = nullptr;
    int rc = validate(cfg, classes, rates, lengths, prices, coef, tg);
    if (rc != QSIM_OK) return rc;
    int ndev = 0;
    CUDA_TRY(cudaGetDeviceCount(&ndev));
    if (ndev < 1) return fail(QSIM_ECUDA, "no CUDA device");
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    qsim *h = new (std::nothrow) qsim();
    if (!h) return fail(QSIM_ENOMEM, "host allocation failed");
    h->device = dev;
    rc = configure(*h, *cfg, classes, prices, coef);
    if (rc != QSIM_OK) { delete h; return rc; }
    Params &p = h->par;
    std::vector<BlockPar> blocks(cfg->nblk);
    fill_blocks(blocks.data(), *cfg, rates, tg);
    cudaError_t e = cudaMalloc(&h->d_blocks, blocks.size() * sizeof(BlockPar));
    if (e == cudaSuccess) e = cudaMemcpy(h->d_blocks, blocks.data(), blocks.size() * sizeof(BlockPar), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && cfg->length_mode == QSIM_LENGTH_TABLE) {
        const std::vector<uint32_t> tab = tables_with_index(lengths, cfg->I);
        e = cudaMalloc(&h->d_lengths, tab.size() * 4);
        if (e == cudaSuccess) e = cudaMemcpy(h->d_lengths, tab.data(), tab.size() * 4, cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = cudaMallocHost(&h->h_flag, 256);
    if (e == cudaSuccess) e = allow_large_smem(reinterpret_cast<const void *>(h->run_fn));
    if (e == cudaSuccess) e = allow_large_smem(reinterpret_cast<const void *>(qsim_init_kernel));
    if (e == cudaSuccess && h->lane_fn) e = allow_large_smem(reinterpret_cast<const void *>(h->lane_fn));
    if (e != cudaSuccess) {
        std::string msg = std::string("device set-up failed: ") + cudaGetErrorString(e);
        qsim_destroy(h);
        return fail(e == cudaErrorMemoryAllocation ? QSIM_ENOMEM : QSIM_ECUDA, msg);
    }
    p.blocks = h->d_blocks;
    p.lengths = h->d_lengths;
    *out = h;
    return QSIM_OK;
}

int qsim_workspace_bytes(const qsim_t *h, size_t *bytes)
{
    if (!h || !bytes) return fail(QSIM_EINVAL, "null argument");
    *bytes = h->sec.total;
    return QSIM_OK;
}

// common part of qsim_bind and qsim_bind_restore: checks the workspace and points the kernel parameters at its sections
static int attach_workspace(qsim_t *h, void *ws, size_t bytes, void *cuda_stream)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    if (!ws) return fail(QSIM_EWORKSPACE, "workspace pointer is null");
    if (bytes < h->sec.total) return fail(QSIM_EWORKSPACE, "workspace too small: need " + std::to_string(h->sec.total) + " bytes");
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return fail(QSIM_EWORKSPACE, "workspace must be 256-byte aligned");
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, ws) != cudaSuccess || (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)) {
        cudaGetLastError();
        return fail(QSIM_EWORKSPACE, "workspace is not device memory");
    }
    h->ws = ws;
    h->stream = static_cast<cudaStream_t>(cuda_stream);
    char *base = static_cast<char *>(ws);
    Params &p = h->par;
    p.hdr = reinterpret_cast<RepHeader *>(base + h->sec.hdr);
    p.srv = base + h->sec.srv;
    p.slot_fin = reinterpret_cast<uint32_t *>(base + h->sec.fin);
    p.slot_rec = reinterpret_cast<SlotRec *>(base + h->sec.rec);
    p.pq = reinterpret_cast<QEntry *>(base + h->sec.pq);
    p.dq = reinterpret_cast<QEntry *>(base + h->sec.dq);
    p.hist_mem = h->cfg.hist ? reinterpret_cast<uint32_t *>(base + h->sec.hist) : nullptr;
    p.not_done = reinterpret_cast<uint32_t *>(base + h->sec.flag);
    p.tarr_g = p.tarr_global ? reinterpret_cast<double *>(base + h->sec.tarr) : nullptr;
    p.pfjob_g = p.tarr_global ? reinterpret_cast<uint32_t *>(base + h->sec.tarr + (size_t)h->cfg.R * h->cfg.N * 8) : nullptr;
    if (p.lane.on) {
        LanePar &q = p.lane;
        q.srv = reinterpret_cast<LaneSrv *>(base + h->sec.l_srv);
        q.tarr = reinterpret_cast<double *>(base + h->sec.l_tarr);
        q.cal_head = reinterpret_cast<uint16_t *>(base + h->sec.l_head);
        q.cal_bm = reinterpret_cast<uint32_t *>(base + h->sec.l_bm);
        q.tree = reinterpret_cast<uint32_t *>(base + h->sec.l_tree);
        q.sfin = reinterpret_cast<uint32_t *>(base + h->sec.l_sfin);
        q.snode = reinterpret_cast<unsigned long long *>(base + h->sec.l_snode);
        q.srec = reinterpret_cast<SlotRec *>(base + h->sec.l_srec);
        q.sfree = reinterpret_cast<uint16_t *>(base + h->sec.l_sfree);
        q.pql = reinterpret_cast<uint32_t *>(base + h->sec.l_pql);
    }
    return QSIM_OK;
}

// Fingerprint of everything that fixes the meaning of the workspace bytes: stored in the workspace at bind, checked when a
// saved workspace is adopted.
static void workspace_tag(const qsim_t *h, unsigned long long tag[2])
{
    const qsim_config &c = h->cfg;
    const unsigned long long words[] = { c.I, c.N, c.R, c.B, c.C, c.nblk, c.gate, c.router, c.placement, c.length_mode, c.qcap, c.hist,
                                         c.seed, c.rep_offset, h->par.Npad, h->par.slots_smem, h->par.srv_bytes, h->par.lane.on,
                                         (unsigned long long)h->sec.total, (unsigned long long)sizeof(RepHeader) };
    unsigned long long x = 0xcbf29ce484222325ull;       // FNV-1a over the bytes of the words
    for (unsigned long long w : words)
        for (int b = 0; b < 8; ++b) { x ^= (w >> (8 * b)) & 0xffull; x *= 0x100000001b3ull; }
    tag[0] = 0x7173696d2d777331ull;                      // "qsim-ws1"
    tag[1] = x;
}

int qsim_bind(qsim_t *h, void *ws, size_t bytes, void *cuda_stream)
{
    int rc = attach_workspace(h, ws, bytes, cuda_stream);
    if (rc != QSIM_OK) return rc;
    {
        unsigned long long tag[2];
        workspace_tag(h, tag);
        CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char *>(h->par.not_done) + 16, tag, sizeof tag, cudaMemcpyHostToDevice, h->stream));
    }
    if (h->par.lane.on) qsim_lane_init_kernel<<<(h->cfg.R + 31u) / 32u, 32, 0, h->stream>>>(h->par);
    else qsim_init_kernel<<<h->cfg.R, 32, h->init_smem, h->stream>>>(h->par);
    CUDA_TRY(cudaGetLastError());
    h->launches++;
    h->bound = true;
    return QSIM_OK;
}

int qsim_bind_restore(qsim_t *h, void *ws, size_t bytes, void *cuda_stream)
{
    int rc = attach_workspace(h, ws, bytes, cuda_stream);
    if (rc != QSIM_OK) return rc;
    // the bytes must come from a handle of the same configuration and layout
    unsigned long long want[2], got[2] = { 0, 0 };
    workspace_tag(h, want);
    CUDA_TRY(cudaMemcpyAsync(got, reinterpret_cast<char *>(h->par.not_done) + 16, sizeof got, cudaMemcpyDeviceToHost, h->stream));
    // the end time reached so far is in every replication's record; a state in which any replication stopped on an
    // internal error cannot be resumed
    std::vector<RepHeader> hdr(h->cfg.R);
    CUDA_TRY(cudaMemcpyAsync(hdr.data(), h->par.hdr, hdr.size() * sizeof(RepHeader), cudaMemcpyDeviceToHost, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    if (got[0] != want[0] || got[1] != want[1])
        return fail(QSIM_ESTATE, "the workspace was not saved by a handle of this configuration");
    for (uint32_t r = 0; r < h->cfg.R; ++r)
        if (hdr[r].err != 0 || !(hdr[r].T_end >= 0.0) || !std::isfinite(hdr[r].T_end))
            return fail(QSIM_ESTATE, "the workspace does not hold a resumable state (replication " + std::to_string(r) + ")");
    // hand-over stamps of chunked launches (qsim_run_kernel) must not repeat a stamp that the saved state still holds
    uint32_t top = 0;
    for (uint32_t r = 0; r < h->cfg.R; ++r) top = std::max(top, hdr[r].seq >> 8);
    h->tag_base = top + 1u;
    const RepHeader &first = hdr[0];
    h->T_end_abs = first.T_end;
    h->bound = true;
    return QSIM_OK;
}

int qsim_run(qsim_t *h, uint64_t horizon_iters)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_run before qsim_bind");
    int rc = launch_run(h, 1u, horizon_iters);
    if (rc != QSIM_OK) return rc;
    // a replication that used up its per-launch event budget is continued by further launches
    for (;;) {
        CUDA_TRY(cudaStreamSynchronize(h->stream));
        bool finished = false;
        rc = launch_outcome(h, finished);
        if (rc != QSIM_OK) return rc;
        if (finished) break;
        rc = launch_run(h, 0u, 0);
        if (rc != QSIM_OK) return rc;
    }
    return QSIM_OK;
}

int qsim_run_until(qsim_t *h, double T)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_run_until before qsim_bind");
    if (!(T >= h->T_end_abs) || !std::isfinite(T)) return fail(QSIM_EINVAL, "end time must be finite and not before the previous one");
    h->T_end_abs = T;
    int rc = launch_run(h, 2u, 0, T);
    if (rc != QSIM_OK) return rc;
    for (;;) {
        CUDA_TRY(cudaStreamSynchronize(h->stream));
        bool finished = false;
        rc = launch_outcome(h, finished);
        if (rc != QSIM_OK) return rc;
        if (finished) break;
        rc = launch_run(h, 0u, 0);
        if (rc != QSIM_OK) return rc;
    }
    return QSIM_OK;
}

int qsim_set_injected(qsim_t *h, const double *t, const uint32_t *job, uint64_t n)
{
    if (!h || !t || !job || n == 0 || n > 0x7fffffffull) return fail(QSIM_EINVAL, "bad injected arrival list");
    if (h->bound) return fail(QSIM_ESTATE, "qsim_set_injected must come before qsim_bind");
    if (h->cfg.nblk != 1) return fail(QSIM_EINVAL, "injected arrivals need nblk == 1");
    if (h->par.lane.on) {
        // trace replay lives in the warp-per-replication family: lay the handle out again for it
        h->allow_lane = false;
        int rc = configure(*h, h->cfg, h->cls, h->prices, h->coef);
        if (rc != QSIM_OK) return rc;
        h->par.blocks = h->d_blocks;
        h->par.lengths = h->d_lengths;
        cudaError_t e = allow_large_smem(reinterpret_cast<const void *>(h->run_fn));
        if (e != cudaSuccess) return fail(QSIM_ECUDA, cudaGetErrorString(e));
    }
    for (uint64_t k = 0; k < n; ++k) {
        if (!(t[k] >= 0.0) || !std::isfinite(t[k]) || (k > 0 && t[k] < t[k - 1])) return fail(QSIM_EINVAL, "injected times must be ascending and >= 0");
        if (job[3 * k] >= h->cfg.I || job[3 * k + 1] < 1 || job[3 * k + 1] > QSIM_LMAX || job[3 * k + 2] < 1 || job[3 * k + 2] > QSIM_LMAX)
            return fail(QSIM_EINVAL, "injected job out of range");
    }
    if (h->d_inject_t) { cudaFree(h->d_inject_t); cudaFree(h->d_inject_job); h->d_inject_t = nullptr; h->d_inject_job = nullptr; }
    CUDA_TRY(cudaMalloc(&h->d_inject_t, n * sizeof(double)));
    CUDA_TRY(cudaMalloc(&h->d_inject_job, n * 3 * sizeof(uint32_t)));
    CUDA_TRY(cudaMemcpy(h->d_inject_t, t, n * sizeof(double), cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(h->d_inject_job, job, n * 3 * sizeof(uint32_t), cudaMemcpyHostToDevice));
    h->par.inject_t = h->d_inject_t;
    h->par.inject_job = h->d_inject_job;
    h->par.n_inject = (uint32_t)n;
    // the trace source lives in the run-time-configured instance
    RunVariant v = pick_run_kernel(h->cfg.N, ~0u);
    if (h->nwarps > 1)
        for (const RunVariant &mw : run_variants())
            if (mw.spl < 0 && (mw.feat & F_GENERIC)) v = mw;
    h->run_fn = v.fn;
    CUDA_TRY(allow_large_smem(reinterpret_cast<const void *>(h->run_fn)));
    return QSIM_OK;
}

int qsim_set_targets(qsim_t *h, const qsim_targets *tg)
{
    if (!h || !tg) return fail(QSIM_EINVAL, "null argument");
    if (h->cfg.nblk != 1) return fail(QSIM_EINVAL, "qsim_set_targets needs nblk == 1");
    if (tg->M > h->cfg.N) return fail(QSIM_EINVAL, "M must be <= N");
    BlockPar bp;
    CUDA_TRY(cudaMemcpyAsync(&bp, h->d_blocks, sizeof bp, cudaMemcpyDeviceToHost, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    bp.M = tg->M;
    for (uint32_t i = 0; i < h->cfg.I; ++i) {
        if (!std::isfinite(tg->xstar[i]) || tg->xstar[i] < 0.0 || !std::isfinite(tg->n_xstar[i]) || !std::isfinite(tg->n_qpstar[i]) ||
            !(tg->p_solo[i] >= 0.0 && tg->p_solo[i] <= 1.0) || !(tg->w_solo[i] >= 0.0) || !std::isfinite(tg->w_solo[i]) ||
            !(tg->w_mix[i] >= 0.0) || !std::isfinite(tg->w_mix[i]))
            return fail(QSIM_EINVAL, "LP targets out of range");
        bp.xstar[i] = tg->xstar[i]; bp.nx[i] = tg->n_xstar[i]; bp.nq[i] = tg->n_qpstar[i]; bp.ps[i] = tg->p_solo[i];
        bp.ws[i] = tg->w_solo[i]; bp.wm[i] = tg->w_mix[i];
    }
    CUDA_TRY(cudaMemcpyAsync(h->d_blocks, &bp, sizeof bp, cudaMemcpyHostToDevice, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    h->targets_changed = true;
    return QSIM_OK;
}

int qsim_set_event_budget(qsim_t *h, uint64_t events_per_launch)
{
    if (!h || events_per_launch == 0) return fail(QSIM_EINVAL, "bad event budget");
    h->par.event_budget = events_per_launch;
    return QSIM_OK;
}

int qsim_sync(qsim_t *h)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    return QSIM_OK;
}

int qsim_layout_info(const qsim_t *h, uint64_t out[4])
{
    if (!h || !out) return fail(QSIM_EINVAL, "null argument");
    out[0] = sizeof(RepHeader);          // bytes per replication copied to the host by qsim_stats
    out[1] = h->par.lane.on ? 0 : h->lay.srv_bytes;   // bytes of per-GPU state staged per replication at kernel entry and exit
    out[2] = h->lay.total;               // shared memory per block
    out[3] = h->nwarps;                  // warps per replication
    return QSIM_OK;
}

int qsim_latency_percentiles(qsim_t *h, const double *q, uint32_t nq, double *ttft, double *tpot)
{
    if (!h || !q || !ttft || !tpot || nq == 0) return fail(QSIM_EINVAL, "null argument");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_latency_percentiles before qsim_bind");
    if (!h->cfg.hist) return fail(QSIM_EINVAL, "percentiles need cfg.hist = 1");
    for (uint32_t k = 0; k < nq; ++k)
        if (!(q[k] > 0.0 && q[k] <= 1.0)) return fail(QSIM_EINVAL, "quantiles must lie in (0, 1]");
    const uint32_t R = h->cfg.R, I = h->cfg.I;
    std::vector<uint32_t> raw((size_t)R * I * 2 * NBIN);
    CUDA_TRY(cudaMemcpyAsync(raw.data(), h->par.hist_mem, raw.size() * 4, cudaMemcpyDeviceToHost, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    std::vector<uint64_t> sum(NBIN);
    for (uint32_t i = 0; i < I; ++i)
        for (int kind = 0; kind < 2; ++kind) {
            std::fill(sum.begin(), sum.end(), 0ull);
            uint64_t total = 0;
            for (uint32_t r = 0; r < R; ++r) {
                const uint32_t *src = raw.data() + (((size_t)r * I + i) * 2 + kind) * NBIN;
                for (int b = 0; b < NBIN; ++b) { sum[b] += src[b]; total += src[b]; }
            }
            double *out = kind == 0 ? ttft : tpot;
            for (uint32_t k = 0; k < nq; ++k) {
                double v = std::nan("");
                if (total > 0) {
                    uint64_t need = (uint64_t)std::ceil(q[k] * (double)total);
                    if (need < 1) need = 1;
                    if (need > total) need = total;
                    uint64_t cum = 0;
                    int b = 0;
                    for (; b < NBIN; ++b) { cum += sum[b]; if (cum >= need) break; }
                    // lower edge of bin b: the double whose top bits are b + ((1023 - 20) << 5)
                    const uint64_t bits = ((uint64_t)b + ((uint64_t)(1023 - 20) << 5)) << 47;
                    std::memcpy(&v, &bits, sizeof v);
                }
                out[(size_t)i * nq + k] = v;
            }
        }
    return QSIM_OK;
}

int qsim_launch_count(const qsim_t *h, uint64_t *launches)
{
    if (!h || !launches) return fail(QSIM_EINVAL, "null argument");
    *launches = h->launches;
    return QSIM_OK;
}

int qsim_round_count(qsim_t *h, uint64_t *rounds)
{
    if (!h || !rounds) return fail(QSIM_EINVAL, "null argument");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_round_count before qsim_bind");
    std::vector<RepHeader> hdr(h->cfg.R);
    CUDA_TRY(cudaMemcpyAsync(hdr.data(), h->par.hdr, hdr.size() * sizeof(RepHeader), cudaMemcpyDeviceToHost, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    uint64_t n = 0;
    for (const RepHeader &H : hdr) n += H.rounds;
    *rounds = n;
    return QSIM_OK;
}

int qsim_reset_stats(qsim_t *h)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_reset_stats before qsim_bind");
    qsim_reset_kernel<<<(h->cfg.R + 127) / 128, 128, 0, h->stream>>>(h->par);
    CUDA_TRY(cudaGetLastError());
    h->launches++;
    return QSIM_OK;
}

int qsim_stats(qsim_t *h, qsim_rep_stats *totals, qsim_rep_stats *per_rep, uint64_t *hist_ttft, uint64_t *hist_tpot)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_stats before qsim_bind");
    const uint32_t R = h->cfg.R, I = h->cfg.I;
    if (!per_rep && !hist_ttft && !hist_tpot) {
        // totals only: reduced on the device, a few KB come back
        if (!totals) { CUDA_TRY(cudaStreamSynchronize(h->stream)); return QSIM_OK; }
        char *base = static_cast<char *>(h->ws);
        TotalsRec *d_out = reinterpret_cast<TotalsRec *>(base + h->sec.red);
        double *d_F = reinterpret_cast<double *>(base + h->sec.red + sizeof(TotalsRecBytes));
        CUDA_TRY(cudaMemsetAsync(d_out, 0, sizeof(TotalsRec), h->stream));
        qsim_totals_gather_kernel<<<(R + 127u) / 128u, 128, 0, h->stream>>>(h->par.hdr, R, I, d_F, d_out);
        qsim_totals_sum_kernel<<<1, 64, 0, h->stream>>>(R, I, d_F, d_out);
        CUDA_TRY(cudaGetLastError());
        h->launches += 2;
        TotalsRec out;
        CUDA_TRY(cudaMemcpyAsync(&out, d_out, sizeof out, cudaMemcpyDeviceToHost, h->stream));
        CUDA_TRY(cudaStreamSynchronize(h->stream));
        if (out.err_code)
            return fail(QSIM_EOVERFLOW, "replication " + std::to_string(out.err_rep) + " hit an internal bound (code " + std::to_string(out.err_code) + ")");
        *totals = out.tot;
        return QSIM_OK;
    }
    std::vector<RepHeader> hdr(R);
    CUDA_TRY(cudaMemcpyAsync(hdr.data(), h->par.hdr, (size_t)R * sizeof(RepHeader), cudaMemcpyDeviceToHost, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    qsim_rep_stats tot;
    std::memset(&tot, 0, sizeof tot);
    for (uint32_t r = 0; r < R; ++r) {
        const RepHeader &H = hdr[r];
        if (H.err) return fail(QSIM_EOVERFLOW, "replication " + std::to_string(r) + " hit an internal bound (code " + std::to_string(H.err) + ")");
        qsim_rep_stats st;
        std::memset(&st, 0, sizeof st);
        rep_stats_of(H, I, st);
        if (per_rep) per_rep[r] = st;
        add_rep_stats(tot, st, I);
    }
    if (totals) *totals = tot;
    if (hist_ttft || hist_tpot) {
        const size_t per = (size_t)I * NBIN;
        if (hist_ttft) std::memset(hist_ttft, 0, (size_t)R * per * 8);
        if (hist_tpot) std::memset(hist_tpot, 0, (size_t)R * per * 8);
        if (h->cfg.hist) {
            std::vector<uint32_t> raw((size_t)R * per * 2);
            CUDA_TRY(cudaMemcpyAsync(raw.data(), h->par.hist_mem, raw.size() * 4, cudaMemcpyDeviceToHost, h->stream));
            CUDA_TRY(cudaStreamSynchronize(h->stream));
            for (uint32_t r = 0; r < R; ++r)
                for (uint32_t i = 0; i < I; ++i)
                    for (uint32_t b = 0; b < NBIN; ++b) {
                        const size_t src = (((size_t)r * I + i) * 2) * NBIN + b;
                        const size_t dst = ((size_t)r * I + i) * NBIN + b;
                        if (hist_ttft) hist_ttft[dst] = raw[src];
                        if (hist_tpot) hist_tpot[dst] = raw[src + NBIN];
                    }
        }
    }
    return QSIM_OK;
}

int qsim_revenue(const qsim_t *h, const qsim_rep_stats *totals, double *bundled_rate, double *separate_rate)
{
    if (!h || !totals) return fail(QSIM_EINVAL, "null argument");
    double tin_done = 0, tin_pf = 0, tout = 0;
    for (uint32_t i = 0; i < h->cfg.I; ++i) {
        tin_done += (double)totals->cls[i].tokens_in_completed;
        tin_pf += (double)totals->cls[i].tokens_in_prefilled;
        tout += (double)totals->cls[i].tokens_out_completed;
    }
    const double denom = (double)h->cfg.N * totals->T_elapsed;
    if (!(denom > 0.0)) return fail(QSIM_ESTATE, "no simulated time has elapsed");
    if (bundled_rate) *bundled_rate = (h->prices[0] * tin_done + h->prices[1] * tout) / denom;
    if (separate_rate) *separate_rate = (h->prices[0] * tin_pf + h->prices[1] * tout) / denom;
    return QSIM_OK;
}

int qsim_server_state(qsim_t *h, uint32_t r, uint32_t *n_dec, uint32_t *it, double *t_next, uint32_t *pf_rem)
{
    if (!h) return fail(QSIM_EINVAL, "null handle");
    if (!h->bound) return fail(QSIM_ESTATE, "qsim_server_state before qsim_bind");
    if (r >= h->cfg.R) return fail(QSIM_EINVAL, "replication index out of range");
    if (h->par.lane.on) {
        std::vector<LaneSrv> rec(h->cfg.N);
        CUDA_TRY(cudaMemcpyAsync(rec.data(), h->par.lane.srv + (size_t)r * h->cfg.N, rec.size() * sizeof(LaneSrv), cudaMemcpyDeviceToHost, h->stream));
        CUDA_TRY(cudaStreamSynchronize(h->stream));
        for (uint32_t g = 0; g < h->cfg.N; ++g) {
            if (n_dec) n_dec[g] = rec[g].ndec;
            if (it) it[g] = rec[g].it;
            if (t_next) t_next[g] = rec[g].tnext;
            if (pf_rem) pf_rem[g] = (rec[g].pfjob >> 31) ? rec[g].pfrem : 0u;
        }
        return QSIM_OK;
    }
    std::vector<char> img(h->lay.srv_bytes);
    CUDA_TRY(cudaMemcpyAsync(img.data(), h->par.srv + (size_t)r * h->lay.srv_bytes, img.size(), cudaMemcpyDeviceToHost, h->stream));
    CUDA_TRY(cudaStreamSynchronize(h->stream));
    const double *tn = reinterpret_cast<const double *>(img.data() + h->lay.off_tnext);
    const uint32_t *itv = reinterpret_cast<const uint32_t *>(img.data() + h->lay.off_it);
    const uint16_t *rem = reinterpret_cast<const uint16_t *>(img.data() + h->lay.off_pfrem);
    const uint16_t *nd = reinterpret_cast<const uint16_t *>(img.data() + h->lay.off_ndec);
    for (uint32_t g = 0; g < h->cfg.N; ++g) {
        if (n_dec) n_dec[g] = nd[g];
        if (it) it[g] = itv[g];
        if (t_next) t_next[g] = tn[g];
        if (pf_rem) pf_rem[g] = rem[g];
    }
    return QSIM_OK;
}

int qsim_destroy(qsim_t *h)
{
    if (!h) return QSIM_OK;
    if (h->bound) cudaStreamSynchronize(h->stream);
    if (h->d_blocks) cudaFree(h->d_blocks);
    if (h->d_lengths) cudaFree(h->d_lengths);
    if (h->d_inject_t) cudaFree(h->d_inject_t);
    if (h->d_inject_job) cudaFree(h->d_inject_job);
    if (h->h_flag) cudaFreeHost(h->h_flag);
    delete h;
    return QSIM_OK;
}

int qsim_simulate(const qsim_config *cfg, const qsim_class *classes, const double *rates, const uint32_t *lengths,
                  const double *prices, const double *coef, const qsim_targets *tg, uint64_t horizon_iters,
                  qsim_rep_stats *totals, qsim_rep_stats *per_rep)
{
    qsim_t *h = nullptr;
    int rc = qsim_create(&h, cfg, classes, rates, lengths, prices, coef, tg);
    if (rc != QSIM_OK) return rc;
    void *ws = nullptr;
    cudaError_t e = cudaMalloc(&ws, h->sec.total);
    if (e != cudaSuccess) {
        qsim_destroy(h);
        return fail(QSIM_ENOMEM, std::string("cudaMalloc(workspace): ") + cudaGetErrorString(e));
    }
    rc = qsim_bind(h, ws, h->sec.total, nullptr);
    if (rc == QSIM_OK) rc = qsim_run(h, horizon_iters);
    if (rc == QSIM_OK) rc = qsim_stats(h, totals, per_rep, nullptr, nullptr);
    const std::string keep = g_err;
    qsim_destroy(h);
    cudaFree(ws);
    if (rc != QSIM_OK) g_err = keep;
    return rc;
}

int qsim_simulate_waves(const qsim_config *cfg, const qsim_class *classes, const double *rates, const uint32_t *lengths,
                        const double *prices, const double *coef, const qsim_targets *tg, uint64_t horizon_iters,
                        uint32_t wave, qsim_rep_stats *totals, qsim_rep_stats *per_rep, uint32_t *waves_run)
{
    int rc = validate(cfg, classes, rates, lengths, prices, coef, tg);
    if (rc != QSIM_OK) return rc;
    const uint32_t R = cfg->R, I = cfg->I;
    // bytes of state for w resident replications (a handle is cheap: it only holds the tables)
    auto bytes_for = [&](uint32_t w, size_t &bytes) -> int {
        qsim_config c = *cfg;
        c.R = w;
        qsim_t *h = nullptr;
        int r = qsim_create(&h, &c, classes, rates, lengths, prices, coef, tg);
        if (r != QSIM_OK) return r;
        bytes = h->sec.total;
        qsim_destroy(h);
        return QSIM_OK;
    };
    uint32_t W = wave == 0 || wave > R ? R : wave;
    size_t need = 0;
    rc = bytes_for(W, need);
    if (rc != QSIM_OK) return rc;
    if (wave == 0) {
        // the largest wave whose state fits in nine tenths of the free device memory
        size_t free_b = 0, total_b = 0;
        CUDA_TRY(cudaMemGetInfo(&free_b, &total_b));
        while (need > free_b / 10 * 9 && W > 1) {
            W = (W + 1) / 2;
            rc = bytes_for(W, need);
            if (rc != QSIM_OK) return rc;
        }
    }
    void *ws = nullptr;
    cudaError_t e = cudaMalloc(&ws, need);
    if (e != cudaSuccess) return fail(QSIM_ENOMEM, std::string("cudaMalloc(workspace of one wave): ") + cudaGetErrorString(e));
    qsim_rep_stats tot;
    std::memset(&tot, 0, sizeof tot);
    std::vector<qsim_rep_stats> buf(per_rep ? 0 : W);
    uint32_t n_waves = 0;
    for (uint32_t done = 0; done < R && rc == QSIM_OK; done += W, ++n_waves) {
        qsim_config c = *cfg;
        c.R = R - done < W ? R - done : W;
        c.rep_offset = cfg->rep_offset + done;        // random streams are keyed by the global replication index
        qsim_t *h = nullptr;
        rc = qsim_create(&h, &c, classes, rates, lengths, prices, coef, tg);
        if (rc != QSIM_OK) break;
        qsim_rep_stats *out = per_rep ? per_rep + done : buf.data();
        if (h->sec.total > need) rc = fail(QSIM_EWORKSPACE, "a later wave needs more state than the first");
        if (rc == QSIM_OK) rc = qsim_bind(h, ws, need, nullptr);
        if (rc == QSIM_OK) rc = qsim_run(h, horizon_iters);
        if (rc == QSIM_OK) rc = qsim_stats(h, nullptr, out, nullptr, nullptr);
        if (rc == QSIM_OK)
            for (uint32_t r = 0; r < c.R; ++r) add_rep_stats(tot, out[r], I);
        const std::string keep = g_err;
        qsim_destroy(h);
        if (rc != QSIM_OK) g_err = keep;
    }
    cudaFree(ws);
    if (rc != QSIM_OK) return rc;
    if (totals) *totals = tot;
    if (waves_run) *waves_run = n_waves;
    return QSIM_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------
// qsim_simulate_static: the whole simulation with no device or pinned-memory allocation (host temporaries only).
// State, tables and the completion flag live in one file-scope device array.  Host code never uses the
// array's name as a pointer: its device address is asked for once per device (cudaGetSymbolAddress).
// ---------------------------------------------------------------------------------------------------
#define QSIM_STATIC_SCRATCH_BYTES (32u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[QSIM_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// device address of the array, per device; written by the first call on a device.  No lock: calls on one device must not
// overlap anyway (they share the array), and two first calls would store the same address.
void *g_static_ptr[kMaxDevices] = {};
}  // namespace

extern "C" int qsim_simulate_static(const qsim_config *cfg, const qsim_class *classes, const double *rates,
                                    const uint32_t *lengths, const double *prices, const double *coef,
                                    const qsim_targets *tg, uint64_t horizon_iters, qsim_rep_stats *totals,
                                    qsim_rep_stats *per_rep, void *cuda_stream)
{
    int rc = validate(cfg, classes, rates, lengths, prices, coef, tg);
    if (rc != QSIM_OK) return rc;
    if (cfg->nblk > 64) return fail(QSIM_EINVAL, "qsim_simulate_static supports at most 64 blocks");
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(QSIM_EINVAL, "device index out of range");
    if (!g_static_ptr[dev]) {
        // first call on this device: resolve the device address of the array (the current device is `dev`)
        void *ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_static_ptr[dev] = ptr;
    }
    char *base = static_cast<char *>(g_static_ptr[dev]);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    qsim h;   // a handle that owns nothing: no table allocation, no pinned flag
    h.allow_lane = false;                  // the built-in scratch is sized for the warp-per-replication layout
    qsim_config nohist = *cfg;
    nohist.hist = 0;                       // histograms are not recorded here
    rc = configure(h, nohist, classes, prices, coef);
    if (rc != QSIM_OK) return rc;
    h.device = dev;
    h.stream = stream;
    h.ws = base;
    Params &p = h.par;
    // scratch = [state sections | block table | length tables]
    const size_t off_blocks = h.sec.total;
    const size_t off_lengths = align256(off_blocks + (size_t)cfg->nblk * sizeof(BlockPar));
    const size_t len_bytes = cfg->length_mode == QSIM_LENGTH_TABLE ? table_bytes(cfg->I) : 0;
    const size_t need = off_lengths + len_bytes;
    if (need > QSIM_STATIC_SCRATCH_BYTES)
        return fail(QSIM_EWORKSPACE, "qsim_simulate_static: this problem needs " + std::to_string(need) +
                                         " bytes of state but the built-in scratch holds " +
                                         std::to_string((size_t)QSIM_STATIC_SCRATCH_BYTES) +
                                         "; reduce R, N*B or qcap, or use qsim_create/qsim_bind with your own workspace");
    BlockPar blocks[64];
    fill_blocks(blocks, *cfg, rates, tg);
    // pageable sources: these copies have returned from the host buffers when the calls return
    CUDA_TRY(cudaMemcpyAsync(base + off_blocks, blocks, (size_t)cfg->nblk * sizeof(BlockPar), cudaMemcpyHostToDevice, stream));
    if (len_bytes) {
        const std::vector<uint32_t> tab = tables_with_index(lengths, cfg->I);
        CUDA_TRY(cudaMemcpyAsync(base + off_lengths, tab.data(), len_bytes, cudaMemcpyHostToDevice, stream));
    }
    p.blocks = reinterpret_cast<const BlockPar *>(base + off_blocks);
    p.lengths = len_bytes ? reinterpret_cast<const uint32_t *>(base + off_lengths) : nullptr;
    p.hdr = reinterpret_cast<RepHeader *>(base + h.sec.hdr);
    p.srv = base + h.sec.srv;
    p.slot_fin = reinterpret_cast<uint32_t *>(base + h.sec.fin);
    p.slot_rec = reinterpret_cast<SlotRec *>(base + h.sec.rec);
    p.pq = reinterpret_cast<QEntry *>(base + h.sec.pq);
    p.dq = reinterpret_cast<QEntry *>(base + h.sec.dq);
    p.hist_mem = nullptr;
    p.not_done = reinterpret_cast<uint32_t *>(base + h.sec.flag);
    p.tarr_g = p.tarr_global ? reinterpret_cast<double *>(base + h.sec.tarr) : nullptr;
    p.pfjob_g = p.tarr_global ? reinterpret_cast<uint32_t *>(base + h.sec.tarr + (size_t)h.cfg.R * h.cfg.N * 8) : nullptr;
    CUDA_TRY(allow_large_smem(reinterpret_cast<const void *>(h.run_fn)));
    CUDA_TRY(allow_large_smem(reinterpret_cast<const void *>(qsim_init_kernel)));
    // the array keeps the previous call's contents: the init kernel rewrites every header and GPU image;
    // queue rings and slot lists are never read before they are written, the flag is cleared per launch
    qsim_init_kernel<<<cfg->R, 32, h.init_smem, stream>>>(p);
    CUDA_TRY(cudaGetLastError());
    bool advance = true;
    for (;;) {
        Params q = p;
        q.advance = advance ? 1u : 0u;
        q.horizon_iters = advance ? horizon_iters : 0;
        CUDA_TRY(cudaMemsetAsync(q.not_done, 0, 4, stream));
        h.run_fn<<<cfg->R, 32 * h.nwarps, h.lay.total, stream>>>(q);
        CUDA_TRY(cudaGetLastError());
        uint32_t left = 0;
        CUDA_TRY(cudaMemcpyAsync(&left, q.not_done, 4, cudaMemcpyDeviceToHost, stream));
        CUDA_TRY(cudaStreamSynchronize(stream));
        if (left == 0) break;
        advance = false;
    }
    h.bound = true;
    rc = qsim_stats(&h, totals, per_rep, nullptr, nullptr);
    h.bound = false;
    return rc;
}

#include "qsim_ctmc.cuh"
