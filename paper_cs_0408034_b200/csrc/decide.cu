// decide_kernel: Broadcast half of the decision table (Sections 1 and 5 of the paper) for short
// candidate lists, with lanes mapped to the process count P.  (The Scatter half has no candidate
// lists and goes through scatter_kernel.)
//
// One CTA owns one table, a group of up to 16 message sizes and a tile of 256 process counts.  All
// four warps work on the same 256 process counts (lane + 32 r, r = 0..7) and split the message
// sizes, so a warp runs on its own from the candidate lists to the staged result and only the
// write-out needs the whole CTA.
//
// Every model of Table 1 is, for a fixed message size (and segment size), a line in P or in
// floor(log2 P):
//     ids 0 1 2 3 4 5:  t = fma(P-1, a, c)           "P list", entries (a, c)
//     ids 7 9:          t = fma(floor(log2 P), a, ceil(log2 P) L)   "log list", entries a
//     ids 6 8:          one cell each, evaluated on their own
// The decision is the lexicographic minimum of (t, id, s) over all cells of all enabled strategies
// (the minimum over s inside a strategy and then over strategies, smallest s and lowest id on
// ties), so one running minimum per process count serves the whole search.  A warp builds the two
// lists of a message size in shared memory (lanes <-> candidates), guesses the winner at the
// process count in the middle of its range (the pilot), starts the running minimum from the
// pilot's cells and takes the pilot out of its list.  Then every cell is evaluated with one DFMA
// and compared with the running minimum on the high 32 bits only, in the integer pipe (times are
// non-negative, so a smaller double never has a larger high word); a group of four list entries in
// which some cell can reach the minimum is re-evaluated with the exact FP64 comparison, for the
// eight-cell rows that need it.  With a good pilot that is rare.
//
// Once started, the running minima (time and winner code) live in shared memory as [m][P], which is
// also the staging layout of the write-out: the loops keep only minus their high words in registers,
// the exact pass reads and writes the minima themselves.  The codes carry the strategy ids as the
// caller names them (OutMap::id_of keeps their order), so the write-out, rows of consecutive m per
// process count, only has to split a code into its id and its segment size.
#include "device_common.cuh"

#include <algorithm>

namespace plogp {

namespace {

constexpr int R = kDecR, U = kDecU;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kStageStride = kDecTileP + 1;  // doubles per staged row: the transposed reads stay conflict-free
constexpr int kCodeStride = kDecTileP + 2;   // 16-bit codes per staged row, for the same reason

constexpr uint32_t kCandNone = 255;   // winner is an unsegmented strategy
constexpr uint32_t kCandWhole = 254;  // segmented winner with no fitting candidate: the whole message
constexpr uint32_t kCodeNever = 0xFFFFu;
constexpr unsigned kNoPilot = 0x1FFu;
constexpr int kIntMax = 0x7FFFFFFF;

struct DecSmem {
    double *tab, *gs, *gm, *lf, *lc, *pm1, *l2, *st_time;
    double2 *l1;
    uint32_t *sval;   // [256]: segment sizes by candidate index; [kCandNone] = 0
    uint16_t *c1, *c2, *st_code;
    int cap1, cap2;
};

__host__ __device__ inline int round_up(int x, int a) { return (x + a - 1) / a * a; }

// Shared-memory layout.  cap1 / cap2: entries of one warp's P list / log list (multiples of U).
__host__ __device__ inline size_t dec_layout(int npad, int n_s, unsigned char *base, DecSmem *o)
{
    const int nsv = n_s > 0 ? n_s : 1;
    const int cap1 = round_up(2 * nsv + 4, U), cap2 = round_up(nsv + 1, U);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += (bytes + 15) & ~size_t(15); return at; };
    const size_t o_tab = take(3 * size_t(npad) * 8), o_gs = take(size_t(nsv) * 8), o_sv = take(256 * 4),
                 o_gm = take(kDecMG * 8), o_lf = take(kDecTileP * 8), o_lc = take(kDecTileP * 8), o_pm = take(kDecTileP * 8),
                 o_l1 = take(size_t(kDecWarps) * cap1 * 16), o_l2 = take(size_t(kDecWarps) * cap2 * 8),
                 o_c1 = take(size_t(kDecWarps) * cap1 * 2), o_c2 = take(size_t(kDecWarps) * cap2 * 2),
                 o_t = take(size_t(kDecMG) * kStageStride * 8), o_c = take(size_t(kDecMG) * kCodeStride * 2);
    if (o) {
        o->tab = reinterpret_cast<double *>(base + o_tab); o->gs = reinterpret_cast<double *>(base + o_gs);
        o->sval = reinterpret_cast<uint32_t *>(base + o_sv); o->gm = reinterpret_cast<double *>(base + o_gm);
        o->lf = reinterpret_cast<double *>(base + o_lf); o->lc = reinterpret_cast<double *>(base + o_lc);
        o->pm1 = reinterpret_cast<double *>(base + o_pm);
        o->l1 = reinterpret_cast<double2 *>(base + o_l1); o->l2 = reinterpret_cast<double *>(base + o_l2);
        o->c1 = reinterpret_cast<uint16_t *>(base + o_c1); o->c2 = reinterpret_cast<uint16_t *>(base + o_c2);
        o->st_time = reinterpret_cast<double *>(base + o_t); o->st_code = reinterpret_cast<uint16_t *>(base + o_c);
        o->cap1 = cap1; o->cap2 = cap2;
    }
    return off;
}

__device__ __forceinline__ int hi32(double x) { return __double2hiint(x); }

// Exact comparison of one cell with the running minimum: (time, code) in lexicographic order, where the code
// orders strategy id first and candidate index (= segment size order) second.
__device__ __forceinline__ void offer(double &bt, uint32_t &bcode, double t, uint32_t code)
{
    if (t <= bt) {
        if (t < bt || code < bcode) { bt = t; bcode = code; }
    }
}

}  // namespace

// ENV: lower-envelope search (DecideParams::envelope), compiled apart so that the exhaustive kernel carries none of it.
template <bool ENV>
__global__ void __launch_bounds__(kDecThreads, 4) decide_kernel(const DecideParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int npad = p.T.npad;
    DecSmem sm;
    dec_layout(npad, p.G.n_s, smem_raw, &sm);
    const uint32_t mask = p.G.mask;

    int b = blockIdx.x;
    const int mgroup = b % p.n_mgroups;
    b /= p.n_mgroups;
    const int ptile = b % p.n_ptiles;
    const int trel = b / p.n_ptiles;
    const int table = p.table0 + trel;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = mgroup * p.mg;  // p.mg <= kDecMG message sizes per CTA (fewer on small grids, for more CTAs)
    const int n_mi = min(p.mg, p.G.n_m - m0);
    const int tile0 = ptile * kDecTileP;
    const int n_valid = min(kDecTileP, p.G.n_P - tile0);

    // g at the kernel's arguments: read from the gap pre-pass where the host has run it, else interpolated here
    const double *grow = p.gaps ? p.gaps + static_cast<size_t>(trel) * p.gaps_stride : nullptr;
    if (!grow) stage_table(sm.tab, p.T, table);
    // floor(log2 P) and ceil(log2 P) of the tile's process counts, as doubles
    for (int i = tid; i < kDecTileP; i += kDecThreads) {
        const int P = P_at(p.G, min(tile0 + i, p.G.n_P - 1));
        sm.lf[i] = static_cast<double>(31 - __clz(P));
        sm.lc[i] = static_cast<double>(32 - __clz(P - 1));
        sm.pm1[i] = static_cast<double>(P - 1);
    }
    __syncthreads();
    const double L = p.T.lat[table];
    for (int si = tid; si < p.G.n_s; si += kDecThreads) {
        const uint32_t s = s_at(p.G, si);
        sm.sval[si] = s;
        sm.gs[si] = grow ? grow[1 + si] : gap_at(sm.tab, npad, static_cast<double>(s));
    }
    if (tid == 0) sm.sval[kCandNone] = 0u;
    if (tid >= kDecThreads - kDecMG) {  // g(m) of the group's message sizes, by the last threads
        const int mi = tid - (kDecThreads - kDecMG);
        if (mi < n_mi) sm.gm[mi] = grow ? grow[1 + p.G.n_s + m0 + mi] : gap_at(sm.tab, npad, static_cast<double>(p.G.m_list[m0 + mi]));
    }
    const double g1 = grow ? grow[0] : gap_at(sm.tab, npad, 1.0);
    const double rdv = 2.0 * g1 + 3.0 * L;  // rendezvous handshake: 2 g(1) + 3 L
    __syncthreads();

    // this thread's cells: process counts at tile offset 32 r + lane; P-1, floor(log2 P) and ceil(log2 P) are read
    // from shared memory where a loop needs them, so that only one of the sets is live at a time
    // the pilot's process count: middle of the tile's valid range
    const int P_mid = P_at(p.G, tile0 + n_valid / 2);
    const double x1_mid = static_cast<double>(P_mid - 1);
    const double x2_mid = static_cast<double>(31 - __clz(P_mid));
    const double c2_mid = static_cast<double>(32 - __clz(P_mid - 1)) * L;

    // the codes carry the strategy ids as the caller names them (the relabelling keeps their order)
    auto idc = [&](int id) { return static_cast<uint32_t>(p.om.id_of[id]) << 8; };
    const uint32_t code2 = idc(2), code5 = idc(5), code9 = idc(9);
    const uint32_t un = mask & 0x1Bu;  // unsegmented members of the P list: ids 0, 1, 3, 4
    const int n_un = __popc(un);
    const bool has2 = (mask >> 2) & 1u, has5 = (mask >> 5) & 1u, has6 = (mask >> 6) & 1u, has7 = (mask >> 7) & 1u,
               has8 = (mask >> 8) & 1u, has9 = (mask >> 9) & 1u;
    // The unsegmented members of the lists do not depend on the message size beyond g(m): lanes 0..3 hold ids 0, 1, 3, 4
    // (Flat Tree (P-1) g + L, its rendezvous form (P-1) g + rdv; Chain (P-1)(g + L), rendezvous (P-1)(g + rdv)) as
    // P-list entries (g(m) + fa, fc), lane 4 the Binomial Tree's log-list entry g(m).
    const int fid = lane < 4 ? lane + (lane >> 1) : 7;
    const bool f_on = lane < 5 && ((mask >> fid) & 1u);
    const int fpos = __popc(un & ((1u << fid) - 1u));
    const double fa = fid == 3 ? L : (fid == 4 ? rdv : 0.0);
    const double fc = fid == 0 ? L : (fid == 1 ? rdv : 0.0);
    const uint16_t fcode = static_cast<uint16_t>(idc(fid) | kCandNone);
    double2 *l1 = sm.l1 + warp * sm.cap1;
    double *l2 = sm.l2 + warp * sm.cap2;
    uint16_t *c1 = sm.c1 + warp * sm.cap1, *c2 = sm.c2 + warp * sm.cap2;

    for (int mi = warp; mi < n_mi; mi += kDecWarps) {
        const int midx = m0 + mi;
        const int ns = p.G.ns_of_m[midx];
        const int nsv = max(ns, 1);  // candidates actually evaluated (none fits: the whole message, k = 1)
        const double gm = sm.gm[mi];
        const double *krow = p.G.k_list + static_cast<size_t>(midx) * p.G.n_s;
        // Lower-envelope search (p.envelope, tables whose gaps never decrease): ids 2 and 9 keep only the candidate
        // with the smallest g(s) k (their minimum over s for every P at once, a rounded fused multiply-add being
        // monotone in it), id 5 only the candidates between its winners at the tile's last and first process
        // count, one more on each side (the lines are sorted by slope g(s) + L, so the winner's index does not
        // grow with P).  Otherwise every candidate enters the lists.
        const bool env = ENV && ns > 0;
        int q_c = 0, lo5 = 0, n5 = nsv;
        if constexpr (ENV) if (env) {
            const double x_first = sm.pm1[0], x_last = sm.pm1[n_valid - 1];
            double qb = CUDART_INF, tf = CUDART_INF, tl = CUDART_INF;
            int qc = kIntMax, ef = kIntMax, el = kIntMax;
            for (int c = lane; c < ns; c += 32) {
                const double gsv = sm.gs[c], k = krow[c];
                const double Q = gsv * k, B = gsv + L, C = gsv * (k - 1.0);
                if (Q < qb) { qb = Q; qc = c; }
                const double t1 = fma(x_first, B, C), t2 = fma(x_last, B, C);
                if (t1 < tf) { tf = t1; ef = c; }
                if (t2 < tl) { tl = t2; el = c; }
            }
            warp_min_pair(qb, qc);
            warp_min_pair(tf, ef);
            warp_min_pair(tl, el);
            q_c = qc;
            lo5 = max(min(ef, el) - 1, 0);
            n5 = min(max(ef, el) + 1, ns - 1) - lo5 + 1;
        }
        const int nq = env ? 1 : nsv;  // entries of ids 2 and 9
        const int o2 = n_un, o5 = o2 + (has2 ? nq : 0), n1 = o5 + (has5 ? n5 : 0);
        const int o9 = has7 ? 1 : 0, n2 = o9 + (has9 ? nq : 0);
        const int n1p = round_up(n1, U), n2p = round_up(n2, U);

        // ---- the two lists of this message size, and each lane's best entry at the pilot's process count ----
        __syncwarp();  // the previous message size's loops have finished reading the lists
        double tb = CUDART_INF;
        unsigned pb = kNoPilot;  // P-list position, or 256 + log-list position
        auto pilot_offer = [&](double t, unsigned pos) {
            if (t < tb) { tb = t; pb = pos; }
        };
        if (f_on) {  // this lane's unsegmented strategy
            if (lane < 4) {
                l1[fpos] = make_double2(gm + fa, fc);
                c1[fpos] = fcode;
                pilot_offer(fma(x1_mid, gm + fa, fc), fpos);
            } else {
                l2[0] = gm;
                c2[0] = fcode;
                pilot_offer(fma(x2_mid, gm, c2_mid), 256u);
            }
        }
        for (int i = n1 + lane; i < n1p; i += 32) {  // padding never reaches the minimum
            l1[i] = make_double2(CUDART_INF, CUDART_INF);
            c1[i] = static_cast<uint16_t>(kCodeNever);
        }
        for (int i = n2 + lane; i < n2p; i += 32) {
            l2[i] = CUDART_INF;
            c2[i] = static_cast<uint16_t>(kCodeNever);
        }
        for (int c = lane; c < nsv; c += 32) {
            // Section 2's k and the line coefficients of Table 1's segmented rows
            double gsv = gm, k = 1.0;
            uint32_t cand = kCandWhole;
            if (ns > 0) {
                gsv = sm.gs[c];
                k = krow[c];  // Section 2's k, from the host's table
                cand = static_cast<uint32_t>(c);
            }
            const double Q = gsv * k;
            const bool in_q = !env || c == q_c, in_5 = !env || (c >= lo5 && c < lo5 + n5);
            const int pq = env ? 0 : c, p5 = env ? c - lo5 : c;  // positions inside the strategies' parts of the lists
            if (has2 && in_q) {  // (P-1) (g(s) k) + L
                l1[o2 + pq] = make_double2(Q, L);
                c1[o2 + pq] = static_cast<uint16_t>(code2 | cand);
                pilot_offer(fma(x1_mid, Q, L), o2 + pq);
            }
            if (has5 && in_5) {  // (P-1) (g(s) + L) + g(s) (k-1)
                const double B = gsv + L, C = gsv * (k - 1.0);
                l1[o5 + p5] = make_double2(B, C);
                c1[o5 + p5] = static_cast<uint16_t>(code5 | cand);
                pilot_offer(fma(x1_mid, B, C), o5 + p5);
            }
            if (has9 && in_q) {  // floor(log2 P) g(s) k + ceil(log2 P) L
                l2[o9 + pq] = Q;
                c2[o9 + pq] = static_cast<uint16_t>(code9 | cand);
                pilot_offer(fma(x2_mid, Q, c2_mid), 256u + o9 + pq);
            }
        }
        // warp-wide pilot: smallest time (high word first, then low word with the position in its last 9 bits)
        const int hmin = __reduce_min_sync(kFull, hi32(tb));
        const unsigned k2 = hi32(tb) == hmin ? ((static_cast<unsigned>(__double2loint(tb)) & ~0x1FFu) | pb) : 0xFFFFFFFFu;
        const unsigned pilot = __reduce_min_sync(kFull, k2) & 0x1FFu;
        __syncwarp();

        double lf[R], lcL[R];  // floor(log2 P); ceil(log2 P), later ceil(log2 P) L
#pragma unroll
        for (int r = 0; r < R; ++r) {
            lf[r] = sm.lf[32 * r + lane];
            lcL[r] = sm.lc[32 * r + lane];
        }

        // ---- running minimum per process count, started from the pilot's cells ----
        double bt[R];
        uint32_t bcode[R];  // strategy id << 8 | candidate index (or kCandNone / kCandWhole)
        if (pilot == kNoPilot) {
#pragma unroll
            for (int r = 0; r < R; ++r) { bt[r] = CUDART_INF; bcode[r] = kCodeNever; }
        } else if (pilot < 256u) {
            const double2 e = l1[pilot];
            const uint32_t code = c1[pilot];
            __syncwarp();
            if (lane == 0) l1[pilot] = make_double2(CUDART_INF, CUDART_INF);
#pragma unroll
            for (int r = 0; r < R; ++r) { bt[r] = fma(sm.pm1[32 * r + lane], e.x, e.y); bcode[r] = code; }
        } else {
            const double a = l2[pilot - 256u];
            const uint32_t code = c2[pilot - 256u];
            __syncwarp();
            if (lane == 0) l2[pilot - 256u] = CUDART_INF;
#pragma unroll
            for (int r = 0; r < R; ++r) { bt[r] = fma(lf[r], a, lcL[r] * L); bcode[r] = code; }
        }
        __syncwarp();

        // one cell per process count (ids 6 and 8): high-word test, exact comparison where it holds
        auto single = [&](uint32_t code, const double *t) {
            int acc = kIntMax;
#pragma unroll
            for (int r = 0; r < R; ++r) acc = min(acc, hi32(t[r]) - hi32(bt[r]));
            if (acc <= 0) {
#pragma unroll
                for (int r = 0; r < R; ++r)
                    if (t[r] < bt[r] || (t[r] == bt[r] && code < bcode[r])) { bt[r] = t[r]; bcode[r] = code; }
            }
        };
        if (has6) {  // Binary Tree (the printed bound): ceil(log2 P) (2 g(m) + L)
            const double w = fma(2.0, gm, L);
            double t[R];
#pragma unroll
            for (int r = 0; r < R; ++r) t[r] = lcL[r] * w;
            single(idc(6) | kCandNone, t);
        }
        if (has8) {  // Binomial Tree Rendezvous: floor(log2 P) g(m) + ceil(log2 P) rdv
            double t[R];
#pragma unroll
            for (int r = 0; r < R; ++r) t[r] = fma(lf[r], gm, lcL[r] * rdv);
            single(idc(8) | kCandNone, t);
        }
        // from here on the running minima live in shared memory (the staging area of the write-out): the loops only need
        // minus their high words, and only the exact pass touches the minima themselves.  (The plain add-then-min form
        // below is left to the compiler on purpose: it splits the work between two pipes and measured faster than the
        // fused add-min instruction.)
        double *st = sm.st_time + mi * kStageStride + lane;
        uint16_t *sc = sm.st_code + mi * kCodeStride + lane;
        int nhb[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            lcL[r] *= L;
            nhb[r] = -hi32(bt[r]);
            st[32 * r] = bt[r];
            sc[32 * r] = static_cast<uint16_t>(bcode[r]);
        }

        // The filter of a group of U list entries: every cell is evaluated (one DFMA each); per process
        // count the smallest high word of the U times minus the high word of the running minimum says
        // whether a cell can reach it (<= 0), and the differences of all R process counts are folded into
        // one minimum, so the test costs integer min / add instructions only (no predicates, no branches)
        // and a single vote decides whether the group needs the exact pass.  The exact pass, (time, id,
        // candidate) in lexicographic order, runs for the rows r that some lane flagged.

        // ---- log list: t = fma(floor(log2 P), a, ceil(log2 P) L) ----
#pragma unroll 1
        for (int j = 0; j < n2p; j += U) {
            const double2 q01 = *reinterpret_cast<const double2 *>(l2 + j), q23 = *reinterpret_cast<const double2 *>(l2 + j + 2);
            int acc = kIntMax;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int h0 = hi32(fma(lf[r], q01.x, lcL[r])), h1 = hi32(fma(lf[r], q01.y, lcL[r]));
                const int h2 = hi32(fma(lf[r], q23.x, lcL[r])), h3 = hi32(fma(lf[r], q23.y, lcL[r]));
                acc = min(acc, min(min(h0, h1), min(h2, h3)) + nhb[r]);
            }
            if (__any_sync(kFull, acc <= 0)) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int h0 = hi32(fma(lf[r], q01.x, lcL[r])), h1 = hi32(fma(lf[r], q01.y, lcL[r]));
                    const int h2 = hi32(fma(lf[r], q23.x, lcL[r])), h3 = hi32(fma(lf[r], q23.y, lcL[r]));
                    if (__any_sync(kFull, min(min(h0, h1), min(h2, h3)) + nhb[r] <= 0)) {
                        double b = st[32 * r];
                        uint32_t code = sc[32 * r];
#pragma unroll 1
                        for (int u = 0; u < U; ++u) offer(b, code, fma(lf[r], l2[j + u], lcL[r]), c2[j + u]);
                        st[32 * r] = b;
                        sc[32 * r] = static_cast<uint16_t>(code);
                        nhb[r] = -hi32(b);
                    }
                }
            }
        }

        // ---- P list: t = fma(P-1, a, c) ----
        double pm1[R];
#pragma unroll
        for (int r = 0; r < R; ++r) pm1[r] = sm.pm1[32 * r + lane];
#pragma unroll 1
        for (int j = 0; j < n1p; j += U) {
            const double2 e0 = l1[j], e1 = l1[j + 1], e2 = l1[j + 2], e3 = l1[j + 3];
            int acc = kIntMax;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int h0 = hi32(fma(pm1[r], e0.x, e0.y)), h1 = hi32(fma(pm1[r], e1.x, e1.y));
                const int h2 = hi32(fma(pm1[r], e2.x, e2.y)), h3 = hi32(fma(pm1[r], e3.x, e3.y));
                acc = min(acc, min(min(h0, h1), min(h2, h3)) + nhb[r]);
            }
            if (__any_sync(kFull, acc <= 0)) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int h0 = hi32(fma(pm1[r], e0.x, e0.y)), h1 = hi32(fma(pm1[r], e1.x, e1.y));
                    const int h2 = hi32(fma(pm1[r], e2.x, e2.y)), h3 = hi32(fma(pm1[r], e3.x, e3.y));
                    if (__any_sync(kFull, min(min(h0, h1), min(h2, h3)) + nhb[r] <= 0)) {
                        double b = st[32 * r];
                        uint32_t code = sc[32 * r];
#pragma unroll 1
                        for (int u = 0; u < U; ++u) {
                            const double2 e = l1[j + u];
                            offer(b, code, fma(pm1[r], e.x, e.y), c1[j + u]);
                        }
                        st[32 * r] = b;
                        sc[32 * r] = static_cast<uint16_t>(code);
                        nhb[r] = -hi32(b);
                    }
                }
            }
        }

    }
    __syncthreads();

    // transposed write-out of the staged group: rows of p.mg consecutive m per process count, running pointers
    if (p.vec_out) {
        // two message sizes per lane: 16-byte, 8-byte and 2-byte stores (the host has checked the alignment)
        const int half = p.mg >> 1;
        const int mi = 2 * (lane & (half - 1)), rows = 32 / half, pr0 = warp * rows + lane / half, prs = kDecWarps * rows;
        if (mi < n_mi) {
            const uint32_t m_u0 = p.G.m_list[m0 + mi], m_u1 = p.G.m_list[m0 + mi + 1];
            const size_t plane = static_cast<size_t>(p.G.n_P) * p.G.n_m;
            const size_t o = (static_cast<size_t>(table - p.out_table0) * p.om.planes + p.om.plane_bcast) * plane +
                             static_cast<size_t>(tile0 + pr0) * p.G.n_m + static_cast<size_t>(m0 + mi);
            const size_t step = static_cast<size_t>(prs) * p.G.n_m;
            double *out_t = p.d_time + o;
            uint32_t *out_s = p.d_sbytes + o;
            uint8_t *out_id = p.d_strategy + o;
            const double *st0 = sm.st_time + mi * kStageStride + pr0, *st1 = st0 + kStageStride;
            const uint16_t *sc0 = sm.st_code + mi * kCodeStride + pr0, *sc1 = sc0 + kCodeStride;
            for (int pr = pr0; pr < n_valid; pr += prs) {
                const uint32_t code0 = *sc0, code1 = *sc1;
                const uint32_t cand0 = code0 & 255u, cand1 = code1 & 255u;
                uint32_t s0 = sm.sval[cand0], s1 = sm.sval[cand1];
                if (cand0 == kCandWhole) s0 = m_u0;
                if (cand1 == kCandWhole) s1 = m_u1;
                *reinterpret_cast<double2 *>(out_t) = make_double2(*st0, *st1);
                *reinterpret_cast<uint2 *>(out_s) = make_uint2(s0, s1);
                *reinterpret_cast<uint16_t *>(out_id) = static_cast<uint16_t>(__byte_perm(code0, code1, 0x0051));
                out_t += step; out_s += step; out_id += step;
                st0 += prs; st1 += prs; sc0 += prs; sc1 += prs;
            }
        }
    } else {
        const int mi = lane & (p.mg - 1), prow = lane / p.mg, rows = 32 / p.mg;
        if (mi < n_mi) {
            const uint32_t m_u = p.G.m_list[m0 + mi];
            const size_t plane = static_cast<size_t>(p.G.n_P) * p.G.n_m;
            const size_t base = (static_cast<size_t>(table - p.out_table0) * p.om.planes + p.om.plane_bcast) * plane + static_cast<size_t>(m0 + mi);
            for (int pr = warp * rows + prow; pr < n_valid; pr += kDecWarps * rows) {
                const size_t o = base + static_cast<size_t>(tile0 + pr) * p.G.n_m;
                const uint32_t code = sm.st_code[mi * kCodeStride + pr];
                const uint32_t cand = code & 255u;
                p.d_time[o] = sm.st_time[mi * kStageStride + pr];
                p.d_strategy[o] = static_cast<uint8_t>(code >> 8);
                p.d_sbytes[o] = cand == kCandWhole ? m_u : sm.sval[cand];
            }
        }
    }
}

size_t decide_smem_bytes(const TableDev &T, const GridDev &G) { return dec_layout(T.npad, G.n_s, nullptr, nullptr); }

template <bool ENV>
static cudaError_t launch_decide_t(const DecideParams &p, size_t smem, unsigned blocks, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024)
        e = cudaFuncSetAttribute(decide_kernel<ENV>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    decide_kernel<ENV><<<blocks, kDecThreads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_decide(const DecideParams &p, cudaStream_t st)
{
    const size_t smem = decide_smem_bytes(p.T, p.G);
    const long long blocks = static_cast<long long>(p.n_mgroups) * p.n_ptiles * p.n_tables_launch;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    return p.envelope ? launch_decide_t<true>(p, smem, static_cast<unsigned>(blocks), st)
                      : launch_decide_t<false>(p, smem, static_cast<unsigned>(blocks), st);
}

}  // namespace plogp
