// Host side of libssd: argument validation, workspace layout, and the segment driver that runs
// Algorithm 1 (forward, storing the state at every segment boundary) and Algorithm 2 (backward,
// segments right to left: recompute from the stored state, back-propagate, hand dh to the left)
// for one SSD layer.  Checkpoint memory is set by the segment length: the scratch holds the chunk
// states of ONE segment, the boundary buffer one state per segment.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

static thread_local int g_last_cuda = 0;

// ---- optional instrumentation: launch counter and per-kernel-kind CUDA-event timing ----
static std::atomic<long long> g_launches{0};
struct ProfEvent { int kind; cudaEvent_t a, b; };
static bool g_prof_on = false;
static std::vector<ProfEvent> g_prof_pool;
static size_t g_prof_used = 0;

static const char *const kKindNames[KIND_COUNT] = {
    "chunk_cumsum", "chunk_state", "state_pass_fwd", "chunk_scan_fwd", "dstate_contrib",
    "state_pass_bwd", "bwd_dx", "bwd_dC", "bwd_dB", "bwd_finish", "reduce_dBdC", "final_dAdD", "glue", "decode_step", "bwd_dBdC", "conv1d", "gated_norm"};

static ProfEvent *prof_begin(int kind, cudaStream_t st) {
    if (!g_prof_on) return nullptr;
    if (g_prof_used == g_prof_pool.size()) {
        ProfEvent ev;
        ev.kind = kind;
        if (cudaEventCreate(&ev.a) != cudaSuccess || cudaEventCreate(&ev.b) != cudaSuccess) return nullptr;
        g_prof_pool.push_back(ev);
    }
    ProfEvent *ev = &g_prof_pool[g_prof_used++];
    ev->kind = kind;
    cudaEventRecord(ev->a, st);
    return ev;
}
static void prof_end(ProfEvent *ev, cudaStream_t st) {
    if (ev) cudaEventRecord(ev->b, st);
}

struct Layout {
    size_t status, cs, dtT, Hst, Hbf, hcarry, Gst, Gbf, gcarry, ghdot, ddt_dir, rho, rho2, psi, psi2, pB, pC, dAp, dDp;
    size_t rhob, psib;
    // second copies (tensor-core path, more than one segment): the state chain of a segment runs on a helper
    // stream while the large kernels of its neighbour still read the first copies
    size_t cs_b, dtT_b, Hbf_b, Gbf_b, rho2_b, ghdot_b;
    // and of what the large kernels of the backward leave for a segment's finishing kernels, so that the next
    // segment's large kernels need not wait for those
    size_t ddt_dir_b, rho_b, rhob_b, psi_b, psib_b, psi2_b, pB_b, pC_b;
    size_t total;
};

// Second copies of the per-segment scratch (and with them the state chain running one segment ahead) pay only when
// there are segments enough to pipeline; with two or three long segments they would cost a third more scratch for
// a per cent or two.
static const int kMinSegmentsForTwins = 4;

struct Plan {
    int B, L, H, P, N, G, Q, seg, nseg, ncs, nct, hpg, nsl, nslf, dtype;
    bool use_tc, serial;
    int64_t x_bs, dt_bs, bc_bs;
    size_t esz;
};

// How many head ranges per group for the tensor-core kernels whose CTAs are (chunk, 128-row block,
// head range).  Half of the CTAs do about 1.8 times the work of the other half (causal structure) and
// are launched first; one CTA per SM, kNumSMs SMs.  The split that minimises the makespan of a greedy
// schedule is taken (cost of a CTA: one head-time of set-up plus its heads).
static int best_head_split(int nchunks, int groups, int batch, int hpg, int max_split) {
    const int kNumSMs = 148;
    // the driver asks once per segment: remember the last few answers
    struct Memo { int nchunks, groups, batch, hpg, max_split, answer; };
    static thread_local Memo memo[4] = {};
    static thread_local int memo_next = 0;
    for (const Memo &m : memo)
        if (m.answer > 0 && m.nchunks == nchunks && m.groups == groups && m.batch == batch && m.hpg == hpg &&
            m.max_split == max_split)
            return m.answer;
    int best = 1;
    double best_t = 1e300;
    for (int ns = 1; ns <= max_split; ++ns) {
        const int hps = (hpg + ns - 1) / ns;
        if ((hpg + hps - 1) / hps != ns) continue;   // would leave an empty range
        double sm[kNumSMs];
        for (int i = 0; i < kNumSMs; ++i) sm[i] = 0.0;
        double makespan = 0.0;
        for (int pass = 0; pass < 2; ++pass)          // all long CTAs, then all short ones
            for (int j = 0; j < nchunks * groups * batch; ++j)
                for (int r = 0; r < ns; ++r) {
                    const int heads = (r == ns - 1) ? hpg - hps * (ns - 1) : hps;
                    const double cost = 1.0 + heads * (pass == 0 ? 1.0 : 0.55);
                    int arg = 0;
                    for (int i = 1; i < kNumSMs; ++i)
                        if (sm[i] < sm[arg]) arg = i;
                    sm[arg] += cost;
                    if (sm[arg] > makespan) makespan = sm[arg];
                }
        if (makespan < best_t - 1e-9) { best_t = makespan; best = ns; }
    }
    memo[memo_next] = Memo{nchunks, groups, batch, hpg, max_split, best};
    memo_next = (memo_next + 1) & 3;
    return best;
}

// Head ranges per group for the fused dB/dC kernel, whose CTAs are (chunk, one of the three causal 128 x 128
// tiles, head range), all of about the same cost: whole waves of 148 CTAs times (one head-time of set-up plus
// the heads of a range), for a reference launch of 16 chunks.  A function of H and G only, so the summation
// order of dB/dC does not depend on the segment length.
static int fused_head_split(int groups, int hpg) {
    int best = 1;
    long best_t = -1;
    const int max_split = hpg >= 4 ? hpg / 4 : 1;
    for (int ns = 1; ns <= max_split; ++ns) {
        const int hps = (hpg + ns - 1) / ns;
        if ((hpg + hps - 1) / hps != ns) continue;
        const long ctas = 16L * 3 * groups * ns;
        const long t = ((ctas + 147) / 148) * (1 + hps);
        if (best_t < 0 || t < best_t) { best_t = t; best = ns; }
    }
    return best;
}

static int make_plan(const ssd_shape_t *s, Plan &pl) {
    if (!s) return SSD_EINVAL;
    if (s->B <= 0 || s->L <= 0 || s->H <= 0 || s->P <= 0 || s->N <= 0 || s->G <= 0 || s->chunk <= 0 ||
        s->seg < 0)
        return SSD_EINVAL;
    if (s->H % s->G) return SSD_EINVAL;
    if (s->dtype != SSD_DTYPE_F32 && s->dtype != SSD_DTYPE_BF16) return SSD_EUNSUPPORTED;
    if (s->P != 64) return SSD_EUNSUPPORTED;
    if (s->N != 64 && s->N != 128) return SSD_EUNSUPPORTED;
    if (s->chunk != 64 && s->chunk != 128 && s->chunk != 256) return SSD_EUNSUPPORTED;
    if (s->L % s->chunk) return SSD_EINVAL;
    const int seg = s->seg == 0 ? s->L : (s->seg > s->L ? s->L : s->seg);
    if (seg % s->chunk) return SSD_EINVAL;
    if (s->x_bstride < 0 || s->dt_bstride < 0 || s->bc_bstride < 0) return SSD_EINVAL;
    pl.B = s->B; pl.L = s->L; pl.H = s->H; pl.P = s->P; pl.N = s->N; pl.G = s->G; pl.Q = s->chunk;
    pl.seg = seg;
    pl.nseg = (s->L + seg - 1) / seg;
    pl.ncs = seg / s->chunk;
    pl.nct = s->L / s->chunk;
    pl.hpg = s->H / s->G;
    pl.dtype = s->dtype;
    pl.esz = s->dtype == SSD_DTYPE_BF16 ? 2 : 4;
    pl.x_bs = s->x_bstride ? s->x_bstride : (int64_t)s->L * s->H * s->P;
    pl.dt_bs = s->dt_bstride ? s->dt_bstride : (int64_t)s->L * s->H;
    pl.bc_bs = s->bc_bstride ? s->bc_bstride : (int64_t)s->L * s->G * s->N;
    if (pl.x_bs < (int64_t)s->L * s->H * s->P || pl.dt_bs < (int64_t)s->L * s->H ||
        pl.bc_bs < (int64_t)s->L * s->G * s->N)
        return SSD_EINVAL;
    if (((size_t)s->H * s->P * pl.esz) % 16 || ((size_t)s->G * s->N * pl.esz) % 16 ||
        ((size_t)pl.x_bs * pl.esz) % 16 || ((size_t)pl.bc_bs * pl.esz) % 16)
        return SSD_EALIGN;
    pl.serial = (s->flags & SSD_FLAG_SERIAL) != 0;
    pl.use_tc = tc_supported(s->dtype, s->flags, s->P, s->N, s->chunk, pl.hpg);
    // Partial slices of the dB/dC head sums.  CUDA-core kernels: one head per slice.  Tensor-core
    // kernels: one slice per CTA head range, chosen for a reference launch of 16 chunks (at least 4
    // heads per range).  A function of H and G only, so the summation order, and with it every bit
    // of dB/dC, is the same for every segment length.
    if (pl.use_tc) {
        pl.nsl = best_head_split(16, pl.G, 1, pl.hpg, pl.hpg >= 4 ? pl.hpg / 4 : 1);
        pl.nslf = fused_head_split(pl.G, pl.hpg);
    } else {
        pl.nsl = pl.hpg;
        pl.nslf = 0;
    }
    return SSD_OK;
}

// `twins`: whether the second copies may exist at all (not for callers that keep every kernel in order on one
// stream: SSD_FLAG_SERIAL and the built-in scratch of ssd_fwd_static_ws).
static void make_layout(const Plan &pl, int op, Layout &lo, bool twins) {
    const size_t PN = (size_t)pl.P * pl.N, BH = (size_t)pl.B * pl.H;
    const size_t vec = BH * pl.ncs * pl.Q * sizeof(float);
    const size_t st = (size_t)pl.B * (pl.ncs + 1) * pl.H * PN;
    const bool bwd = (op == SSD_OP_BWD_SEG);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
    memset(&lo, 0, sizeof(lo));
    lo.status = take(256);
    lo.cs = take(vec);
    lo.dtT = take(vec);
    lo.Hst = take(st * sizeof(float));
    lo.Hbf = take(pl.use_tc ? st * 2 : 0);
    lo.hcarry = take(BH * PN * sizeof(float));
    const bool twin = twins && pl.use_tc && pl.nseg >= kMinSegmentsForTwins;
    lo.cs_b = take(twin ? vec : 0);
    lo.dtT_b = take(twin ? vec : 0);
    lo.Hbf_b = take(twin ? st * 2 : 0);
    if (bwd) {
        lo.Gst = take(st * sizeof(float));
        lo.Gbf = take(pl.use_tc ? st * 2 : 0);
        lo.gcarry = take(BH * PN * sizeof(float));
        lo.ghdot = take(BH * pl.ncs * 16 * sizeof(float));
        lo.ddt_dir = take(vec);
        lo.rho = take(vec);
        lo.rho2 = take(pl.use_tc ? vec : 0);
        lo.psi = take(vec);
        lo.psi2 = take(vec);
        const int slots = (2 * pl.nslf > pl.nsl) ? 2 * pl.nslf : pl.nsl;   // fused kernel: two slots per head range
        const size_t part = (size_t)pl.B * pl.seg * pl.G * slots * pl.N * sizeof(float);
        lo.pB = take(part);
        lo.pC = take(part);
        lo.dAp = take(BH * pl.nct * sizeof(float));
        lo.dDp = take(BH * pl.nct * 16 * sizeof(float));
        lo.Gbf_b = take(twin ? st * 2 : 0);
        lo.rho2_b = take(twin ? vec : 0);
        lo.ghdot_b = take(twin ? BH * pl.ncs * 16 * sizeof(float) : 0);
        lo.rhob = take(pl.use_tc ? vec : 0);
        lo.psib = take(pl.use_tc ? vec : 0);
        lo.ddt_dir_b = take(twin ? vec : 0);
        lo.rho_b = take(twin ? vec : 0);
        lo.rhob_b = take(twin ? vec : 0);
        lo.psi_b = take(twin ? vec : 0);
        lo.psib_b = take(twin ? vec : 0);
        lo.psi2_b = take(twin ? vec : 0);
        lo.pB_b = take(twin ? part : 0);
        lo.pC_b = take(twin ? part : 0);
    }
    lo.total = o;
}

static bool misaligned(const void *p) { return ((uintptr_t)p & 15u) != 0; }

static int check_device() {
    static thread_local int cached_dev = -1;
    static thread_local int cached_ok = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_last_cuda = (int)e; return SSD_ECUDA; }
    if (dev != cached_dev) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) { g_last_cuda = (int)e; return SSD_ECUDA; }
        cached_dev = dev;
        cached_ok = (major == 10);
    }
    return cached_ok ? SSD_OK : SSD_EDEVICE;
}

// Helper streams per (host thread, device) with the events that fork them off the caller's stream and join them
// back: s[4] recomputes a segment's chunk states (in the forward: the whole state chain is on s[0]), s[0] runs the
// state-gradient part of the chain, s[1] / s[3] the dB/dC kernel of even / odd segments beside dx on the caller's
// stream, s[2] a segment's two finishing kernels.  Created on first use, never
// destroyed (they hold no device memory); the caller's stream stays the only one the caller has to order
// against.  Events indexed [2] alternate with the segment, like the second copies of the scratch regions.
struct SideStreams {
    int dev = -1;
    cudaStream_t s[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};   // gradient chain | dB/dC, even | tails | dB/dC, odd | recompute
    cudaEvent_t start = nullptr;
    cudaEvent_t chain_done[2] = {nullptr, nullptr}, big_done[2] = {nullptr, nullptr}, tail_done[2] = {nullptr, nullptr};
    cudaEvent_t rec_done[2] = {nullptr, nullptr}, join[2] = {nullptr, nullptr}, dx_done[2] = {nullptr, nullptr};
};
static SideStreams *side_streams() {
    static thread_local std::vector<SideStreams> all;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    for (auto &a : all)
        if (a.dev == dev) return &a;
    SideStreams a;
    a.dev = dev;
    for (int i = 0; i < 5; ++i)
        if (cudaStreamCreateWithFlags(&a.s[i], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    cudaEvent_t *evs[] = {&a.start, &a.chain_done[0], &a.chain_done[1], &a.big_done[0], &a.big_done[1], &a.tail_done[0],
                          &a.tail_done[1], &a.rec_done[0], &a.rec_done[1], &a.join[0], &a.join[1], &a.dx_done[0], &a.dx_done[1]};
    for (cudaEvent_t *ev : evs)
        if (cudaEventCreateWithFlags(ev, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    all.push_back(a);
    return &all.back();
}

#define SSD_TRY(expr)                                   \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) {                       \
            g_last_cuda = (int)e__;                     \
            return SSD_ECUDA;                           \
        }                                               \
    } while (0)

// one kernel launch of kind `kind` on stream `st`
#define SSD_LAUNCH(kind, expr)                          \
    do {                                                \
        ProfEvent *pe__ = prof_begin(kind, st);         \
        cudaError_t e__ = (expr);                       \
        prof_end(pe__, st);                             \
        g_launches.fetch_add(1, std::memory_order_relaxed); \
        if (e__ != cudaSuccess) {                       \
            g_last_cuda = (int)e__;                     \
            return SSD_ECUDA;                           \
        }                                               \
    } while (0)

static void fill_params(const Plan &pl, const Layout &lo, void *ws, SegParams &sp) {
    memset(&sp, 0, sizeof(sp));
    sp.B = pl.B; sp.L = pl.L; sp.H = pl.H; sp.P = pl.P; sp.N = pl.N; sp.G = pl.G; sp.Q = pl.Q;
    sp.hpg = pl.hpg; sp.ncs = pl.ncs; sp.nct = pl.nct; sp.nsl = pl.nsl;
    sp.ndd = pl.use_tc ? 8 : pl.Q / 64;
    sp.x_bs = pl.x_bs; sp.dt_bs = pl.dt_bs; sp.bc_bs = pl.bc_bs;
    char *w = (char *)ws;
    sp.status = (unsigned int *)(w + lo.status);
    sp.cs = (float *)(w + lo.cs);
    sp.dtT = (float *)(w + lo.dtT);
    sp.Hst = (float *)(w + lo.Hst);
    sp.Hbf = (__nv_bfloat16 *)(w + lo.Hbf);
    sp.hcarry = (float *)(w + lo.hcarry);
    sp.Gst = (float *)(w + lo.Gst);
    sp.Gbf = (__nv_bfloat16 *)(w + lo.Gbf);
    sp.gcarry = (float *)(w + lo.gcarry);
    sp.ghdot = (float *)(w + lo.ghdot);
    sp.ddt_dir = (float *)(w + lo.ddt_dir);
    sp.rho = (float *)(w + lo.rho);
    sp.rho2 = nullptr;   // set by the backward driver on the tensor-core path
    sp.psi = (float *)(w + lo.psi);
    sp.psi2 = (float *)(w + lo.psi2);
    sp.pB = (float *)(w + lo.pB);
    sp.pC = (float *)(w + lo.pC);
    sp.dAp = (float *)(w + lo.dAp);
    sp.dDp = (float *)(w + lo.dDp);
}

static void set_segment(const Plan &pl, int k, SegParams &sp) {
    sp.t0 = k * pl.seg;
    const int len = (pl.L - sp.t0 < pl.seg) ? pl.L - sp.t0 : pl.seg;
    sp.nc = len / pl.Q;
    sp.c0 = sp.t0 / pl.Q;
    // Head ranges per group for the scan kernels (at least two heads per CTA so the shared score tile
    // is reused).  Their outputs are per head, so this choice cannot change any result bit.
    sp.nsplit_scan = best_head_split(sp.nc, pl.G, pl.B, pl.hpg, pl.hpg >= 2 ? pl.hpg / 2 : 1);
}

// Points the kernels at the first or the second copy of the scratch regions that exist twice.
static void select_copy(const Layout &lo, void *ws, bool second, bool bwd, SegParams &sp) {
    char *w = (char *)ws;
    sp.cs = (float *)(w + (second ? lo.cs_b : lo.cs));
    sp.dtT = (float *)(w + (second ? lo.dtT_b : lo.dtT));
    sp.Hbf = (__nv_bfloat16 *)(w + (second ? lo.Hbf_b : lo.Hbf));
    if (bwd) {
        sp.Gbf = (__nv_bfloat16 *)(w + (second ? lo.Gbf_b : lo.Gbf));
        sp.rho2 = (float *)(w + (second ? lo.rho2_b : lo.rho2));
        sp.ghdot = (float *)(w + (second ? lo.ghdot_b : lo.ghdot));
        sp.ddt_dir = (float *)(w + (second ? lo.ddt_dir_b : lo.ddt_dir));
        sp.rho = (float *)(w + (second ? lo.rho_b : lo.rho));
        sp.psi = (float *)(w + (second ? lo.psi_b : lo.psi));
        sp.psi2 = (float *)(w + (second ? lo.psi2_b : lo.psi2));
        sp.pB = (float *)(w + (second ? lo.pB_b : lo.pB));
        sp.pC = (float *)(w + (second ? lo.pC_b : lo.pC));
        if (sp.rhob) {   // the fused dB/dC kernel is in use
            sp.rhob = (float *)(w + (second ? lo.rhob_b : lo.rhob));
            sp.psib = (float *)(w + (second ? lo.psib_b : lo.psib));
        }
    }
}

static int forward_impl(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                        const void *Bm, const void *Cm, const float *D, const float *h0, void *y,
                        float *h_final, float *boundary, bool need_boundary, void *ws,
                        size_t ws_bytes, void *stream, bool may_use_helper_stream = true) {
    Plan pl;
    int rc = make_plan(shape, pl);
    if (rc) return rc;
    if (!x || !dt || !A || !Bm || !Cm || !D || !y || !ws) return SSD_EINVAL;
    if (need_boundary && !boundary) return SSD_EINVAL;
    if (misaligned(x) || misaligned(dt) || misaligned(A) || misaligned(Bm) || misaligned(Cm) ||
        misaligned(D) || misaligned(y) || (h0 && misaligned(h0)) || (h_final && misaligned(h_final)) ||
        (boundary && misaligned(boundary)))
        return SSD_EALIGN;
    Layout lo;
    make_layout(pl, need_boundary ? SSD_OP_FWD_SEG : SSD_OP_FWD, lo, may_use_helper_stream && !pl.serial);
    if (((uintptr_t)ws & 255u) || ws_bytes < lo.total) return SSD_EWORKSPACE;
    rc = check_device();
    if (rc) return rc;

    cudaStream_t st = (cudaStream_t)stream;
    SegParams sp;
    fill_params(pl, lo, ws, sp);
    sp.x = x; sp.dt = dt; sp.A = A; sp.Bm = Bm; sp.Cm = Cm; sp.D = D; sp.y = y;
    SSD_TRY(cudaMemsetAsync(sp.status, 0, 256, st));
    TcMaps maps;
    if (pl.use_tc && !tc_make_maps(sp, maps)) return SSD_ECUDA;
    const long long PN = (long long)pl.P * pl.N;
    if (pl.use_tc && pl.nseg >= kMinSegmentsForTwins && may_use_helper_stream && !pl.serial && !g_prof_on) {
        // Algorithm 1 with the state chain one segment ahead: chunk states and state pass of segment k run on a
        // helper stream while the caller's stream still computes y of segment k-1, whose last, partly idle wave
        // they fill.  What both touch (cumulative sums, dt per chunk, bf16 chunk states) exists twice and
        // alternates; the fp32 chunk sums and the carried state belong to the chain alone.
        SideStreams *side = side_streams();
        if (!side) { g_last_cuda = (int)cudaGetLastError(); return SSD_ECUDA; }
        TcMaps maps_b;
        select_copy(lo, ws, true, false, sp);
        if (!tc_make_maps(sp, maps_b)) return SSD_ECUDA;
        cudaStream_t chain = side->s[0];
        SSD_TRY(cudaEventRecord(side->start, st));
        SSD_TRY(cudaStreamWaitEvent(chain, side->start, 0));
        for (int k = 0; k < pl.nseg; ++k) {
            const int par = k & 1;
            set_segment(pl, k, sp);
            select_copy(lo, ws, par != 0, false, sp);
            const TcMaps &mk = par ? maps_b : maps;
            if (k >= 2) SSD_TRY(cudaStreamWaitEvent(chain, side->big_done[par], 0));   // y of segment k-2 has read this copy
            {
                cudaStream_t st = chain;
                SSD_LAUNCH(KIND_CHUNK_STATE, launch_chunk_state_tc(sp, mk, STATE_MODE_FWD, st));
                const float *init = (k == 0) ? h0 : sp.hcarry;
                float *bnd = boundary ? boundary + (size_t)k * pl.H * PN : nullptr;
                SSD_LAUNCH(KIND_STATE_PASS_FWD, launch_state_pass_fwd(sp, init, (long long)pl.H * PN, bnd, (long long)pl.nseg * pl.H * PN,
                                              (k == pl.nseg - 1) ? h_final : nullptr, true, st));
                SSD_TRY(cudaEventRecord(side->chain_done[par], st));
            }
            SSD_TRY(cudaStreamWaitEvent(st, side->chain_done[par], 0));
            SSD_LAUNCH(KIND_SCAN_FWD, launch_scan_tc(sp, mk, SC_FWD, st));
            if (k + 2 < pl.nseg) SSD_TRY(cudaEventRecord(side->big_done[par], st));
        }
        return SSD_OK;
    }
    for (int k = 0; k < pl.nseg; ++k) {
        set_segment(pl, k, sp);
        if (pl.use_tc) {   // the tensor-core chunk-state kernel computes the chunk cumsum itself
            SSD_LAUNCH(KIND_CHUNK_STATE, launch_chunk_state_tc(sp, maps, STATE_MODE_FWD, st));
        } else {
            SSD_LAUNCH(KIND_CUMSUM, launch_chunk_cumsum(sp, st));
            SSD_LAUNCH(KIND_CHUNK_STATE, launch_chunk_state_simt(sp, pl.dtype, STATE_MODE_FWD, st));
        }
        const float *init = (k == 0) ? h0 : sp.hcarry;
        float *bnd = boundary ? boundary + (size_t)k * pl.H * PN : nullptr;
        SSD_LAUNCH(KIND_STATE_PASS_FWD, launch_state_pass_fwd(sp, init, (long long)pl.H * PN, bnd, (long long)pl.nseg * pl.H * PN,
                                      (k == pl.nseg - 1) ? h_final : nullptr, pl.use_tc, st));
        if (pl.use_tc) SSD_LAUNCH(KIND_SCAN_FWD, launch_scan_tc(sp, maps, SC_FWD, st));
        else SSD_LAUNCH(KIND_SCAN_FWD, launch_masked_product_simt(sp, pl.dtype, MP_FWD, st));
    }
    return SSD_OK;
}

// ---- self-test of the bounded device-side wait: a barrier that nothing ever arrives on
// One warp waits on it with the given limit, gives up, records that in the status word and returns normally: the
// same mbar_wait path, status word and host read-back that every kernel of the library relies on, with no copy in
// flight and no tensor memory held, so that giving up is harmless here.
__global__ void k_selftest_wait(unsigned int *status, long long limit_clk, long long *waited_clk) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        sm100::mbar_init(&bar, 1);
        abort_flag = 0;
        sm100::fence_barrier_init();
    }
    __syncthreads();
    const long long t0 = clock64();
    const bool done = sm100::mbar_wait_limited(&bar, 0, &abort_flag, status, limit_clk);
    if (threadIdx.x == 0 && waited_clk) *waited_clk = done ? -1 : clock64() - t0;
}

// ---- built-in scratch for ssd_fwd_static_ws (callers that cannot allocate) ----
// Lives in the device image of this library: one copy per GPU that loads it, for the life of the
// process.  In host code `g_static_ws` is only a handle for cudaGetSymbolAddress, never a pointer.
static __device__ __align__(256) unsigned char g_static_ws[SSD_STATIC_WS_BYTES];

static const int kMaxDevices = 64;
static std::mutex g_static_mu;
static void *g_static_addr[kMaxDevices] = {nullptr};

// Device address of g_static_ws on the current device, looked up once per device.
static int static_ws_address(void **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_last_cuda = (int)e; return SSD_ECUDA; }
    if (dev < 0 || dev >= kMaxDevices) return SSD_EDEVICE;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_ws);
        if (e != cudaSuccess || !ptr) { g_last_cuda = (int)e; return SSD_ECUDA; }
        g_static_addr[dev] = ptr;
    }
    *out = g_static_addr[dev];
    return SSD_OK;
}

}  // namespace ssd

using namespace ssd;

extern "C" {

size_t ssd_workspace_bytes(const ssd_shape_t *shape, int op) {
    Plan pl;
    if (make_plan(shape, pl)) return 0;
    if (op != SSD_OP_FWD && op != SSD_OP_FWD_SEG && op != SSD_OP_BWD_SEG) return 0;
    Layout lo;
    make_layout(pl, op, lo, !pl.serial);
    return lo.total;
}

size_t ssd_boundary_bytes(const ssd_shape_t *shape) {
    Plan pl;
    if (make_plan(shape, pl)) return 0;
    return (size_t)pl.B * pl.nseg * pl.H * pl.P * pl.N * sizeof(float);
}

int ssd_fwd(const ssd_shape_t *shape, const void *x, const float *dt, const float *A, const void *Bm,
            const void *Cm, const float *D, const float *h0, void *y, float *h_final, void *ws,
            size_t ws_bytes, void *stream) {
    return forward_impl(shape, x, dt, A, Bm, Cm, D, h0, y, h_final, nullptr, false, ws, ws_bytes, stream);
}

int ssd_fwd_static_ws(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                      const void *Bm, const void *Cm, const float *D, const float *h0, void *y,
                      float *h_final, void *stream) {
    Plan pl;
    int rc = make_plan(shape, pl);
    if (rc) return rc;
    Layout lo;
    make_layout(pl, SSD_OP_FWD, lo, false);      // in order on one stream: no second copies
    if (lo.total > (size_t)SSD_STATIC_WS_BYTES) return SSD_ETOOLARGE;
    if (!x || !dt || !A || !Bm || !Cm || !D || !y) return SSD_EINVAL;
    rc = check_device();
    if (rc) return rc;
    void *ws = nullptr;
    rc = static_ws_address(&ws);
    if (rc) return rc;
    // forward_impl zeroes the status word on the stream and writes every other scratch region
    // before reading it, so stale contents of the shared array cannot leak into the outputs.
    return forward_impl(shape, x, dt, A, Bm, Cm, D, h0, y, h_final, nullptr, false, ws,
                        (size_t)SSD_STATIC_WS_BYTES, stream, false);
}

int ssd_fwd_segmented(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                      const void *Bm, const void *Cm, const float *D, const float *h0, void *y,
                      float *h_final, float *boundary, void *ws, size_t ws_bytes, void *stream) {
    return forward_impl(shape, x, dt, A, Bm, Cm, D, h0, y, h_final, boundary, true, ws, ws_bytes, stream);
}

int ssd_bwd_segmented(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                      const void *Bm, const void *Cm, const float *D, const float *boundary,
                      const void *dy, const float *dh_final, void *dx, float *ddt, float *dA, void *dB,
                      void *dC, float *dD, float *dh0, void *ws, size_t ws_bytes, void *stream) {
    Plan pl;
    int rc = make_plan(shape, pl);
    if (rc) return rc;
    if (!x || !dt || !A || !Bm || !Cm || !D || !boundary || !dy || !dx || !ddt || !dA || !dB || !dC ||
        !dD || !ws)
        return SSD_EINVAL;
    if (misaligned(x) || misaligned(dt) || misaligned(A) || misaligned(Bm) || misaligned(Cm) ||
        misaligned(D) || misaligned(boundary) || misaligned(dy) || (dh_final && misaligned(dh_final)) ||
        misaligned(dx) || misaligned(ddt) || misaligned(dA) || misaligned(dB) || misaligned(dC) ||
        misaligned(dD) || (dh0 && misaligned(dh0)))
        return SSD_EALIGN;
    Layout lo;
    make_layout(pl, SSD_OP_BWD_SEG, lo, !pl.serial);
    if (((uintptr_t)ws & 255u) || ws_bytes < lo.total) return SSD_EWORKSPACE;
    rc = check_device();
    if (rc) return rc;

    cudaStream_t st = (cudaStream_t)stream;
    SegParams sp;
    fill_params(pl, lo, ws, sp);
    sp.x = x; sp.dt = dt; sp.A = A; sp.Bm = Bm; sp.Cm = Cm; sp.D = D; sp.dy = dy;
    sp.dx = dx; sp.ddt = ddt; sp.dB = dB; sp.dC = dC;
    sp.dx_skip = (shape->flags & SSD_FLAG_SKIP_GRAD) ? 1.f : 0.f;
    if (pl.use_tc) sp.rho2 = (float *)((char *)ws + lo.rho2);
    SSD_TRY(cudaMemsetAsync(sp.status, 0, 256, st));
    TcMaps maps;
    if (pl.use_tc && !tc_make_maps(sp, maps)) return SSD_ECUDA;
    const long long PN = (long long)pl.P * pl.N;
    const bool fused_bc = pl.use_tc && !(shape->flags & SSD_FLAG_SPLIT_BC);
    if (fused_bc) {
        sp.nsl = pl.nslf;
        sp.bc_fused = 1;
        sp.rhob = (float *)((char *)ws + lo.rhob);
        sp.psib = (float *)((char *)ws + lo.psib);
    }
    SideStreams *side = nullptr;
    if (pl.use_tc && !(shape->flags & SSD_FLAG_SERIAL) && !g_prof_on) {
        side = side_streams();
        if (!side) { g_last_cuda = (int)cudaGetLastError(); return SSD_ECUDA; }
    }
    if (side) {
        // Algorithm 2 as three pipelines that meet through events.  Segment k (right to left) needs
        //   chain(k): Recompute_Forward (chunk states, forward state pass), the state-gradient contributions and
        //             the backward state pass -- all it takes from segment k+1 is the state gradient handed left;
        //   big(k)  : dx on the caller's stream beside dB/dC on a second one -- they read what chain(k) left;
        //   tail(k) : the two short finishing kernels.
        // chain(k-1) runs on its own stream while big(k) is busy and fills the SMs that big(k)'s last, partly
        // idle wave leaves free; tail(k) runs under big(k-1)'s predecessors likewise.  What chain(k-1) writes and
        // big(k) / tail(k) read exists twice and alternates with the segment (cumulative sums, dt per chunk, both
        // bf16 state copies, rho2, <G,H>); the fp32 chunk sums and the carried gradient belong to the chain alone.
        const bool twin = pl.nseg >= kMinSegmentsForTwins;    // else one copy: chain(k) then also waits for tail(k+1)
        TcMaps maps_b;
        if (twin) {
            select_copy(lo, ws, true, true, sp);
            if (!tc_make_maps(sp, maps_b)) return SSD_ECUDA;
        }
        cudaStream_t grads = side->s[0], recomp = side->s[4], tails = side->s[2];
        SSD_TRY(cudaEventRecord(side->start, st));
        SSD_TRY(cudaStreamWaitEvent(recomp, side->start, 0));
        SSD_TRY(cudaStreamWaitEvent(grads, side->start, 0));
        int par = 0;
        for (int k = pl.nseg - 1; k >= 0; --k) {
            par = twin ? ((pl.nseg - 1 - k) & 1) : 0;
            set_segment(pl, k, sp);
            select_copy(lo, ws, par != 0, true, sp);
            const TcMaps &mk = par ? maps_b : maps;
            // ---- chain(k), first half: Recompute_Forward.  Its copy was last read by big(k+2) and tail(k+2) (of k+1
            // when there is one copy only); the fp32 chunk sums belong to this stream alone.
            if (k + (twin ? 2 : 1) <= pl.nseg - 1) SSD_TRY(cudaStreamWaitEvent(recomp, side->tail_done[par], 0));
            {
                cudaStream_t st = recomp;
                SSD_LAUNCH(KIND_CHUNK_STATE, launch_chunk_state_tc(sp, mk, STATE_MODE_FWD, st));
                SSD_LAUNCH(KIND_STATE_PASS_FWD, launch_state_pass_fwd(sp, boundary + (size_t)k * pl.H * PN, (long long)pl.nseg * pl.H * PN,
                                              nullptr, 0, nullptr, true, st));
                SSD_TRY(cudaEventRecord(side->rec_done[par], st));
            }
            // ---- chain(k), second half: the state gradients, which alone wait for segment k+1 (stream order: the
            // gradient handed left, and the fp32 contributions that belong to this stream alone)
            SSD_TRY(cudaStreamWaitEvent(grads, side->rec_done[par], 0));
            {
                cudaStream_t st = grads;
                SSD_LAUNCH(KIND_DSTATE, launch_chunk_state_tc(sp, mk, STATE_MODE_DSTATE, st));
                const float *ginit = (k == pl.nseg - 1) ? dh_final : sp.gcarry;
                float *gleft = (k == 0 && dh0) ? dh0 : sp.gcarry;
                SSD_LAUNCH(KIND_STATE_PASS_BWD, launch_state_pass_bwd(sp, ginit, gleft, true, st));
                SSD_TRY(cudaEventRecord(side->chain_done[par], st));
            }
            // ---- big(k); what it leaves for tail(k) (direct ddt, rho, psi, partial dB/dC slices) alternates too, and
            // chain(k) has already waited for tail(k+2), the last reader of this copy.  The dB/dC kernels of
            // neighbouring segments are on different streams: with short segments one alone does not fill the GPU.
            cudaStream_t bcs = side->s[par ? 3 : 1];
            SSD_TRY(cudaStreamWaitEvent(st, side->chain_done[par], 0));
            SSD_TRY(cudaStreamWaitEvent(bcs, side->chain_done[par], 0));
            {
                cudaStream_t st = bcs;
                if (fused_bc) {
                    SSD_LAUNCH(KIND_BWD_DBDC, launch_grad_bc_fused(sp, mk, st));
                } else {
                    SSD_LAUNCH(KIND_BWD_DC, launch_grad_bc_tc(sp, mk, GB_DC, st));
                    SSD_LAUNCH(KIND_BWD_DB, launch_grad_bc_tc(sp, mk, GB_DB, st));
                }
                SSD_TRY(cudaEventRecord(side->join[par], st));
            }
            SSD_LAUNCH(KIND_BWD_DX, launch_scan_tc(sp, mk, SC_DX, st));
            SSD_TRY(cudaEventRecord(side->dx_done[par], st));
            // ---- tail(k), after both
            SSD_TRY(cudaStreamWaitEvent(tails, side->dx_done[par], 0));
            SSD_TRY(cudaStreamWaitEvent(tails, side->join[par], 0));
            {
                cudaStream_t st = tails;
                SSD_LAUNCH(KIND_BWD_FINISH, launch_bwd_finish(sp, st));
                SSD_LAUNCH(KIND_REDUCE_DBDC, launch_reduce_dbdc(sp, pl.dtype, st));
                SSD_TRY(cudaEventRecord(side->tail_done[par], st));
            }
        }
        SSD_TRY(cudaStreamWaitEvent(st, side->tail_done[par], 0));   // the finishing stream is in order: this covers every segment
    } else {
        for (int k = pl.nseg - 1; k >= 0; --k) {
            set_segment(pl, k, sp);
            // Recompute_Forward: chunk-entry states of segment k from the stored boundary state
            if (pl.use_tc) {   // the tensor-core chunk-state kernel computes the chunk cumsum itself
                SSD_LAUNCH(KIND_CHUNK_STATE, launch_chunk_state_tc(sp, maps, STATE_MODE_FWD, st));
            } else {
                SSD_LAUNCH(KIND_CUMSUM, launch_chunk_cumsum(sp, st));
                SSD_LAUNCH(KIND_CHUNK_STATE, launch_chunk_state_simt(sp, pl.dtype, STATE_MODE_FWD, st));
            }
            SSD_LAUNCH(KIND_STATE_PASS_FWD, launch_state_pass_fwd(sp, boundary + (size_t)k * pl.H * PN, (long long)pl.nseg * pl.H * PN,
                                          nullptr, 0, nullptr, pl.use_tc, st));
            // Backward through the segment; dh enters from the right, leaves to the left
            if (pl.use_tc) SSD_LAUNCH(KIND_DSTATE, launch_chunk_state_tc(sp, maps, STATE_MODE_DSTATE, st));
            else SSD_LAUNCH(KIND_DSTATE, launch_chunk_state_simt(sp, pl.dtype, STATE_MODE_DSTATE, st));
            const float *ginit = (k == pl.nseg - 1) ? dh_final : sp.gcarry;
            float *gleft = (k == 0 && dh0) ? dh0 : sp.gcarry;
            SSD_LAUNCH(KIND_STATE_PASS_BWD, launch_state_pass_bwd(sp, ginit, gleft, pl.use_tc, st));
            if (pl.use_tc) SSD_LAUNCH(KIND_BWD_DX, launch_scan_tc(sp, maps, SC_DX, st));
            else SSD_LAUNCH(KIND_BWD_DX, launch_masked_product_simt(sp, pl.dtype, MP_BWD_DX, st));
            if (fused_bc) {
                SSD_LAUNCH(KIND_BWD_DBDC, launch_grad_bc_fused(sp, maps, st));
            } else if (pl.use_tc) {
                SSD_LAUNCH(KIND_BWD_DC, launch_grad_bc_tc(sp, maps, GB_DC, st));
                SSD_LAUNCH(KIND_BWD_DB, launch_grad_bc_tc(sp, maps, GB_DB, st));
            } else {
                SSD_LAUNCH(KIND_BWD_DC, launch_masked_product_simt(sp, pl.dtype, MP_DC, st));
                SSD_LAUNCH(KIND_BWD_DB, launch_masked_product_simt(sp, pl.dtype, MP_DB, st));
            }
            SSD_LAUNCH(KIND_BWD_FINISH, launch_bwd_finish(sp, st));
            SSD_LAUNCH(KIND_REDUCE_DBDC, launch_reduce_dbdc(sp, pl.dtype, st));
        }
    }
    SSD_LAUNCH(KIND_FINAL, launch_final_dAdD(sp, dA, dD, (shape->flags & SSD_FLAG_ACCUM_PARAM_GRADS) != 0, st));
    return SSD_OK;
}

static int glue_check(const ssd_shape_t *s, const void *a, const void *b, size_t &esz, long long &bs) {
    if (!s || !a || !b) return SSD_EINVAL;
    if (s->B <= 0 || s->L <= 0 || s->H <= 0) return SSD_EINVAL;
    if (s->P != 64) return SSD_EUNSUPPORTED;
    if (s->dtype != SSD_DTYPE_F32 && s->dtype != SSD_DTYPE_BF16) return SSD_EUNSUPPORTED;
    esz = s->dtype == SSD_DTYPE_BF16 ? 2 : 4;
    bs = s->x_bstride ? s->x_bstride : (long long)s->L * s->H * s->P;
    if (bs < (long long)s->L * s->H * s->P) return SSD_EINVAL;
    if (misaligned(a) || misaligned(b) || ((size_t)bs * esz) % 16) return SSD_EALIGN;
    return SSD_OK;
}

int ssd_glue_fwd(const ssd_shape_t *shape, const void *x, const void *y, const float *W, void *x_next, void *stream) {
    size_t esz; long long bs;
    int rc = glue_check(shape, x, y, esz, bs);
    if (rc) return rc;
    if (!W || !x_next) return SSD_EINVAL;
    if (misaligned(W) || misaligned(x_next)) return SSD_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_GLUE, launch_glue(shape->dtype, false, x, y, W, x_next, (long long)shape->L * shape->H, bs, shape->B, st));
    return SSD_OK;
}

int ssd_glue_bwd(const ssd_shape_t *shape, const void *g_next, const float *W, void *dz, void *stream) {
    size_t esz; long long bs;
    int rc = glue_check(shape, g_next, dz, esz, bs);
    if (rc) return rc;
    if (!W) return SSD_EINVAL;
    if (misaligned(W)) return SSD_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_GLUE, launch_glue(shape->dtype, true, g_next, nullptr, W, dz, (long long)shape->L * shape->H, bs, shape->B, st));
    return SSD_OK;
}

int ssd_glue_residual(const ssd_shape_t *shape, void *dx, const void *dz, void *stream) {
    size_t esz; long long bs;
    int rc = glue_check(shape, dx, dz, esz, bs);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_GLUE, launch_residual(shape->dtype, dx, dz, (long long)shape->L * shape->H * shape->P, bs, shape->B, st));
    return SSD_OK;
}

int ssd_decode_step(const ssd_shape_t *s, const void *x, const float *dt, const float *A, const void *Bm,
                    const void *Cm, const float *D, float *h, void *y, void *stream) {
    if (!s || !x || !dt || !A || !Bm || !Cm || !D || !h || !y) return SSD_EINVAL;
    if (s->B <= 0 || s->L != 1 || s->H <= 0 || s->P <= 0 || s->G <= 0 || s->H % s->G) return SSD_EINVAL;
    if (s->N != 64 && s->N != 128) return SSD_EUNSUPPORTED;
    if (s->dtype != SSD_DTYPE_F32 && s->dtype != SSD_DTYPE_BF16) return SSD_EUNSUPPORTED;
    const long long x_bs = s->x_bstride ? s->x_bstride : (long long)s->H * s->P;
    const long long dt_bs = s->dt_bstride ? s->dt_bstride : (long long)s->H;
    const long long bc_bs = s->bc_bstride ? s->bc_bstride : (long long)s->G * s->N;
    if (x_bs < (long long)s->H * s->P || dt_bs < s->H || bc_bs < (long long)s->G * s->N) return SSD_EINVAL;
    if (misaligned(x) || misaligned(dt) || misaligned(A) || misaligned(Bm) || misaligned(Cm) || misaligned(D) ||
        misaligned(h) || misaligned(y))
        return SSD_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_DECODE, launch_decode_step(s->dtype, s->N, x, dt, A, Bm, Cm, D, h, y, s->B, s->H, s->P, s->G,
                                               x_bs, dt_bs, bc_bs, st));
    return SSD_OK;
}

static int conv_check(int B, int L, int C, int dtype, long long &bs, long long u_bstride) {
    if (B <= 0 || L < 3 || C <= 0 || (C % 8)) return SSD_EINVAL;
    if (dtype != SSD_DTYPE_F32 && dtype != SSD_DTYPE_BF16) return SSD_EUNSUPPORTED;
    bs = u_bstride ? u_bstride : (long long)L * C;
    if (bs < (long long)L * C) return SSD_EINVAL;
    if (((size_t)bs * (dtype == SSD_DTYPE_BF16 ? 2 : 4)) % 16) return SSD_EALIGN;
    return SSD_OK;
}

size_t ssd_conv_workspace_bytes(int B, int L, int C) {
    if (B <= 0 || L <= 0 || C <= 0) return 0;
    return (size_t)B * conv_tiles(L) * 5 * C * sizeof(float);
}

int ssd_conv_fwd(int B, int L, int C, int dtype, const void *u, long long u_bstride, const float *w, const float *bias,
                 const void *state_in, void *out, void *state_out, void *stream) {
    long long bs;
    int rc = conv_check(B, L, C, dtype, bs, u_bstride);
    if (rc) return rc;
    if (!u || !w || !bias || !out) return SSD_EINVAL;
    if (misaligned(u) || misaligned(w) || misaligned(bias) || misaligned(out) || (state_in && misaligned(state_in)) ||
        (state_out && misaligned(state_out)))
        return SSD_EALIGN;
    rc = check_device();
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_CONV, launch_conv_fwd(dtype, u, bs, w, bias, state_in, out, state_out, B, L, C, st));
    return SSD_OK;
}

int ssd_conv_bwd(int B, int L, int C, int dtype, const void *u, long long u_bstride, const float *w, const float *bias,
                 const void *state_in, const void *dout, const float *dtail, void *du, float *dstate, float *dw,
                 float *dbias, int accumulate, void *ws, size_t ws_bytes, void *stream) {
    long long bs;
    int rc = conv_check(B, L, C, dtype, bs, u_bstride);
    if (rc) return rc;
    if (!u || !w || !bias || !dout || !du || !dw || !dbias || !ws) return SSD_EINVAL;
    if (misaligned(u) || misaligned(w) || misaligned(bias) || misaligned(dout) || misaligned(du) || misaligned(dw) ||
        misaligned(dbias) || (state_in && misaligned(state_in)) || (dtail && misaligned(dtail)) ||
        (dstate && misaligned(dstate)))
        return SSD_EALIGN;
    if (((uintptr_t)ws & 255u) || ws_bytes < ssd_conv_workspace_bytes(B, L, C)) return SSD_EWORKSPACE;
    rc = check_device();
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_CONV, launch_conv_bwd(dtype, u, bs, w, bias, state_in, dout, dtail, du, dstate, dw, dbias,
                                          accumulate ? 1 : 0, (float *)ws, B, L, C, st));
    return SSD_OK;
}

static int norm_check(long long rows, int D, int group, int dtype) {
    if (rows <= 0 || D <= 0 || group <= 0 || (D % group) || (group % 4)) return SSD_EINVAL;
    if (group > gated_norm_max_group() || gated_norm_tiles(rows) > 2147483647ll || D / group > 65535) return SSD_EUNSUPPORTED;
    if (dtype != SSD_DTYPE_F32 && dtype != SSD_DTYPE_BF16) return SSD_EUNSUPPORTED;
    if (((size_t)D * (dtype == SSD_DTYPE_BF16 ? 2 : 4)) % 16) return SSD_EALIGN;
    return SSD_OK;
}

size_t ssd_gated_norm_workspace_bytes(long long rows, int D) {
    if (rows <= 0 || D <= 0) return 0;
    return (size_t)gated_norm_tiles(rows) * D * sizeof(float);
}

int ssd_gated_norm_fwd(long long rows, int D, int group, int dtype, const void *y, const void *z, const float *gamma, float eps,
                       void *out, void *stream) {
    int rc = norm_check(rows, D, group, dtype);
    if (rc) return rc;
    if (!y || !z || !gamma || !out) return SSD_EINVAL;
    if (misaligned(y) || misaligned(z) || misaligned(gamma) || misaligned(out)) return SSD_EALIGN;
    rc = check_device();
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_NORM, launch_gated_norm_fwd(dtype, y, z, gamma, eps, out, rows, D, group, st));
    return SSD_OK;
}

int ssd_gated_norm_bwd(long long rows, int D, int group, int dtype, const void *y, const void *z, const float *gamma, float eps,
                       const void *dout, void *dy, void *dz, float *dgamma, int accumulate, void *ws, size_t ws_bytes,
                       void *stream) {
    int rc = norm_check(rows, D, group, dtype);
    if (rc) return rc;
    if (!y || !z || !gamma || !dout || !dy || !dz || !dgamma || !ws) return SSD_EINVAL;
    if (misaligned(y) || misaligned(z) || misaligned(gamma) || misaligned(dout) || misaligned(dy) || misaligned(dz) ||
        misaligned(dgamma))
        return SSD_EALIGN;
    if (((uintptr_t)ws & 255u) || ws_bytes < ssd_gated_norm_workspace_bytes(rows, D)) return SSD_EWORKSPACE;
    rc = check_device();
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_LAUNCH(KIND_NORM, launch_gated_norm_bwd(dtype, y, z, gamma, eps, dout, dy, dz, dgamma, accumulate ? 1 : 0, (float *)ws,
                                                rows, D, group, st));
    return SSD_OK;
}

int ssd_selftest_wait_timeout(void *ws, size_t ws_bytes, long long limit_cycles, void *stream) {
    if (!ws || limit_cycles < 0) return SSD_EINVAL;
    if (((uintptr_t)ws & 255u) || ws_bytes < 512) return SSD_EWORKSPACE;
    int rc = check_device();
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    SSD_TRY(cudaMemsetAsync(ws, 0, 512, st));
    k_selftest_wait<<<1, 32, 0, st>>>((unsigned int *)ws, limit_cycles, (long long *)((char *)ws + 256));
    SSD_TRY(cudaGetLastError());
    return SSD_OK;
}

int ssd_poll_status(void *ws) {
    if (!ws) return SSD_EINVAL;
    unsigned int word = 0;
    cudaError_t e = cudaMemcpy(&word, ws, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { g_last_cuda = (int)e; return SSD_ECUDA; }
    return word ? SSD_ETIMEOUT : SSD_OK;
}

const char *ssd_strerror(int code) {
    switch (code) {
        case SSD_OK: return "ok";
        case SSD_EINVAL: return "invalid argument (null pointer, bad size, H % G, L % chunk or seg % chunk)";
        case SSD_EUNSUPPORTED: return "unsupported shape or dtype (P=64, N in {64,128}, chunk in {64,128,256})";
        case SSD_EALIGN: return "pointer or stride not 16-byte aligned";
        case SSD_EWORKSPACE: return "workspace too small or not 256-byte aligned";
        case SSD_EDEVICE: return "current device is not compute capability 10.x";
        case SSD_ECUDA: return "CUDA call failed (see ssd_last_cuda_error)";
        case SSD_ETIMEOUT: return "a bounded device-side wait expired";
        case SSD_ETOOLARGE: return "shape needs more scratch than the built-in static buffer (SSD_STATIC_WS_BYTES); reduce seg or pass your own workspace to ssd_fwd";
        default: return "unknown error";
    }
}

int ssd_version(void) { return SSD_VERSION; }

long long ssd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int ssd_kernel_kinds(void) { return KIND_COUNT; }

const char *ssd_kernel_name(int kind) {
    return (kind >= 0 && kind < KIND_COUNT) ? kKindNames[kind] : "";
}

int ssd_profile(int enable) {
    g_prof_on = enable != 0;
    g_prof_used = 0;
    return SSD_OK;
}

int ssd_profile_read(double *ms, long long *launches, int n) {
    if (!ms || !launches || n < KIND_COUNT) return SSD_EINVAL;
    for (int i = 0; i < n; ++i) { ms[i] = 0.0; launches[i] = 0; }
    for (size_t i = 0; i < g_prof_used; ++i) {
        ProfEvent &ev = g_prof_pool[i];
        cudaError_t e = cudaEventSynchronize(ev.b);
        float t = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t, ev.a, ev.b);
        if (e != cudaSuccess) { g_last_cuda = (int)e; return SSD_ECUDA; }
        ms[ev.kind] += (double)t;
        launches[ev.kind] += 1;
    }
    g_prof_used = 0;
    return SSD_OK;
}

int ssd_last_cuda_error(void) { return g_last_cuda; }

}  // extern "C"
