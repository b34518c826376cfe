// segmin_kernel: the segment-size search of Section 3.1 for plogp_predict on short candidate lists, with lanes
// mapped to the process count P: for each segmented strategy of Table 1 (ids 2, 5, 9) on its own, the minimum
// of the model over the candidate segment sizes and the smallest size that attains it.
//
// Same building blocks as decide_kernel (decide.cu), with one running minimum per strategy instead of one
// over all of them.  One CTA (8 warps) owns one table, 16 consecutive message sizes (two per warp) and a tile
// of 256 process counts (lane + 32 r, r = 0..7).  For a fixed message size the models are lines,
//     id 2: fma(P-1, Q, L)      id 9: fma(floor(log2 P), Q, ceil(log2 P) L)      Q = g(s) k
//     id 5: fma(P-1, B, C)      B = g(s) + L, C = g(s) (k-1)
// so a warp first builds the coefficient lists of its message sizes (lanes <-> candidates); then the CTA takes
// one strategy at a time: every warp sweeps that strategy's list for its message sizes, the results are staged
// in shared memory as [m][P], and the whole CTA writes the strategy's plane out as rows of 16 consecutive m
// (128-byte row segments) before the next strategy reuses the staging area.  In a sweep
// every cell is evaluated with one DFMA and compared with the running minimum on the high
// 32 bits only, in the integer pipe (times are non-negative); a group of four candidates in which some cell
// can reach the minimum is re-evaluated with the exact comparison, (time, candidate) in lexicographic order,
// for the rows of 32 process counts that need it.  The running minima start from a pilot: for ids 2 and 9 the
// candidate with the smallest Q, which is their winner for every P (the sweep still visits every cell), for
// id 5 the winner at the tile's middle process count.  The outputs are the prediction planes
// time[table][13][P][m] and best_s[table][3][P][m].
#include "device_common.cuh"

#include <algorithm>
#include <type_traits>

namespace plogp {

namespace {

constexpr int R = kSegR, U = 4;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kIntMax = 0x7FFFFFFF;
constexpr int kStride = kSegTileP + 1;   // doubles per staged row: the transposed reads stay conflict-free
constexpr int kIStride = kSegTileP + 2;  // 16-bit candidate indices per staged row
constexpr uint32_t kWhole = 0xFFFEu;     // no candidate fits: the whole message in one segment
static_assert(kMaxInlineS <= 64, "warp_argmin_pilot keeps a candidate index in six bits");

struct SegSmem {
    double *tab, *gs, *gm, *lf, *lc, *pm1, *lq, *qp, *st_time;
    double2 *l5, *ep;
    uint32_t *sval;
    uint16_t *st_idx;
    int *pc;
    int cap;
};

__host__ __device__ inline size_t seg_layout(int npad, int n_s, unsigned char *base, SegSmem *o)
{
    const int nsv = n_s > 0 ? n_s : 1;
    const int cap = (nsv + U - 1) / U * U;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += (bytes + 15) & ~size_t(15); return at; };
    const size_t o_tab = take(3 * size_t(npad) * 8), o_gs = take(size_t(nsv) * 8), o_sv = take(size_t(nsv) * 4),
                 o_gm = take(kSegMG * 8), o_lf = take(kSegTileP * 8), o_lc = take(kSegTileP * 8), o_pm = take(kSegTileP * 8),
                 o_lq = take(size_t(kSegMG) * cap * 8), o_l5 = take(size_t(kSegMG) * cap * 16),
                 o_qp = take(kSegMG * 8), o_ep = take(kSegMG * 16), o_pc = take(2 * kSegMG * 4),
                 o_t = take(size_t(kSegMG) * kStride * 8), o_i = take(size_t(kSegMG) * kIStride * 2);
    if (o) {
        o->tab = reinterpret_cast<double *>(base + o_tab); o->gs = reinterpret_cast<double *>(base + o_gs);
        o->sval = reinterpret_cast<uint32_t *>(base + o_sv); o->gm = reinterpret_cast<double *>(base + o_gm);
        o->lf = reinterpret_cast<double *>(base + o_lf); o->lc = reinterpret_cast<double *>(base + o_lc);
        o->pm1 = reinterpret_cast<double *>(base + o_pm);
        o->lq = reinterpret_cast<double *>(base + o_lq); o->l5 = reinterpret_cast<double2 *>(base + o_l5);
        o->qp = reinterpret_cast<double *>(base + o_qp); o->ep = reinterpret_cast<double2 *>(base + o_ep);
        o->pc = reinterpret_cast<int *>(base + o_pc);
        o->st_time = reinterpret_cast<double *>(base + o_t); o->st_idx = reinterpret_cast<uint16_t *>(base + o_i);
        o->cap = cap;
    }
    return off;
}

__device__ __forceinline__ int hi32(double x) { return __double2hiint(x); }

// Index (< 64) of a smallest non-negative value over the warp, up to the last 6 bits of its low word: two integer
// warp reductions (high word, then low word with the index in its last bits).  Good enough for a pilot: the sweep's
// exact comparisons settle what the pilot leaves open.
__device__ __forceinline__ int warp_argmin_pilot(double v, int idx)
{
    const int hmin = __reduce_min_sync(0xffffffffu, hi32(v));
    const unsigned key = hi32(v) == hmin ? ((static_cast<unsigned>(__double2loint(v)) & ~0x3Fu) | static_cast<unsigned>(idx & 0x3F)) : 0xFFFFFFFFu;
    return static_cast<int>(__reduce_min_sync(0xffffffffu, key) & 0x3Fu);
}

__device__ __forceinline__ void offer(double &bt, uint32_t &bidx, double t, uint32_t idx)
{
    if (t <= bt) {
        if (t < bt || idx < bidx) { bt = t; bidx = idx; }
    }
}

}  // namespace

__global__ void __launch_bounds__(kSegThreads, 2) segmin_kernel(const SegminParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int npad = p.T.npad;
    SegSmem sm;
    seg_layout(npad, p.G.n_s, smem_raw, &sm);
    const uint32_t mask = p.G.mask;

    int b = blockIdx.x;
    const int mgroup = b % p.n_mgroups;
    b /= p.n_mgroups;
    const int ptile = b % p.n_ptiles;
    const int trel = b / p.n_ptiles;
    const int table = p.table0 + trel;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = mgroup * kSegMG;
    const int n_mi = min(kSegMG, p.G.n_m - m0);
    const int tile0 = ptile * kSegTileP;
    const int n_valid = min(kSegTileP, p.G.n_P - tile0);

    // g at the kernel's arguments: read from the gap pre-pass where the host has run it, else interpolated here
    const double *grow = p.gaps ? p.gaps + static_cast<size_t>(trel) * p.gaps_stride : nullptr;
    if (!grow) stage_table(sm.tab, p.T, table);
    for (int i = tid; i < kSegTileP; i += kSegThreads) {
        const int P = P_at(p.G, min(tile0 + i, p.G.n_P - 1));
        sm.lf[i] = static_cast<double>(31 - __clz(P));
        sm.lc[i] = static_cast<double>(32 - __clz(P - 1));
        sm.pm1[i] = static_cast<double>(P - 1);
    }
    __syncthreads();
    const double L = p.T.lat[table];
    for (int si = tid; si < p.G.n_s; si += kSegThreads) {
        const uint32_t s = s_at(p.G, si);
        sm.sval[si] = s;
        sm.gs[si] = grow ? grow[1 + si] : gap_at(sm.tab, npad, static_cast<double>(s));
    }
    if (tid >= kSegThreads - kSegMG) {
        const int mi = tid - (kSegThreads - kSegMG);
        if (mi < n_mi) sm.gm[mi] = grow ? grow[1 + p.G.n_s + m0 + mi] : gap_at(sm.tab, npad, static_cast<double>(p.G.m_list[m0 + mi]));
    }
    __syncthreads();

    const double x_mid = sm.pm1[n_valid / 2];

    // ---- phase 0: the coefficient lists of the warp's message sizes (lanes <-> candidates) and the pilots ----
    for (int mi = warp; mi < n_mi; mi += kSegWarps) {
        const int midx = m0 + mi;
        const int ns = p.G.ns_of_m[midx];
        const int nsv = max(ns, 1);  // candidates actually evaluated (none fits: the whole message, k = 1)
        const int np = (nsv + U - 1) / U * U;
        const double gm = sm.gm[mi];
        const double *krow = p.G.k_list + static_cast<size_t>(midx) * p.G.n_s;
        double *lq = sm.lq + mi * sm.cap;
        double2 *l5 = sm.l5 + mi * sm.cap;
        double qb = CUDART_INF, tb = CUDART_INF;
        int qc = kIntMax, tc = kIntMax;
        for (int c = lane; c < np; c += 32) {
            double Q = CUDART_INF, B = CUDART_INF, C = CUDART_INF;  // padding never reaches a minimum
            if (c < nsv) {
                double gsv = gm, k = 1.0;
                if (ns > 0) {
                    gsv = sm.gs[c];
                    k = krow[c];  // Section 2's k, from the host's table
                }
                Q = gsv * k;
                B = gsv + L;
                C = gsv * (k - 1.0);
                if (Q < qb) { qb = Q; qc = c; }
                const double t = fma(x_mid, B, C);
                if (t < tb) { tb = t; tc = c; }
            }
            lq[c] = Q;
            l5[c] = make_double2(B, C);
        }
        qc = warp_argmin_pilot(qb, qc);  // smallest Q: the winner of ids 2 and 9 for every P
        tc = warp_argmin_pilot(tb, tc);  // id 5's winner at the middle of the tile
        __syncwarp();
        // the pilots leave the lists (their own cells would always pass the filter); the running minima start from them
        const double q_pilot = lq[qc];
        const double2 e_pilot = l5[tc];
        __syncwarp();
        if (lane == 0) {
            lq[qc] = CUDART_INF;
            l5[tc] = make_double2(CUDART_INF, CUDART_INF);
            sm.qp[mi] = q_pilot; sm.ep[mi] = e_pilot;
            sm.pc[2 * mi] = qc; sm.pc[2 * mi + 1] = tc;
        }
    }
    __syncwarp();  // the lists and pilots of a message size are read by the warp that wrote them

    const size_t plane = static_cast<size_t>(p.G.n_P) * p.G.n_m;
    const int ids[3] = {2, 5, 9};
    // ---- one strategy at a time: every warp sweeps it for its message sizes, then the CTA writes the plane ----
#pragma unroll 1
    for (int q = 0; q < 3; ++q) {
        if (!((mask >> ids[q]) & 1u)) continue;
        for (int mi = warp; mi < n_mi; mi += kSegWarps) {
            const int midx = m0 + mi;
            const int ns = p.G.ns_of_m[midx];
            const int np = (max(ns, 1) + U - 1) / U * U;
            const double *lq = sm.lq + mi * sm.cap;
            const double2 *l5 = sm.l5 + mi * sm.cap;
            const uint32_t whole = ns > 0 ? 0u : 1u;
            auto stage = [&](const double *bt, const uint32_t *bidx) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    sm.st_time[mi * kStride + 32 * r + lane] = bt[r];
                    sm.st_idx[mi * kIStride + 32 * r + lane] = static_cast<uint16_t>(whole ? kWhole : bidx[r]);
                }
            };
            // Filter of a group of U candidates: the smallest high word of the U times minus the high word of the running
            // minimum says whether a cell can reach it (<= 0); the differences of all R process counts are folded into one
            // integer minimum and one vote decides whether the group needs the exact pass.
            auto sweep_q = [&](auto is9_tag) {
                constexpr bool IS9 = decltype(is9_tag)::value;
                // id 2: fma(P-1, Q, L); id 9: fma(floor(log2 P), Q, ceil(log2 P) L)
                const double q_pilot = sm.qp[mi];
                const int qc = sm.pc[2 * mi];
                double x[R], c9[IS9 ? R : 1];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    x[r] = IS9 ? sm.lf[32 * r + lane] : sm.pm1[32 * r + lane];
                    if (IS9) c9[r] = sm.lc[32 * r + lane] * L;
                }
                if (!IS9) c9[0] = L;
                double bt[R];
                uint32_t bidx[R];
#pragma unroll
                for (int r = 0; r < R; ++r) { bt[r] = fma(x[r], q_pilot, c9[IS9 ? r : 0]); bidx[r] = static_cast<uint32_t>(qc); }
#pragma unroll 1
                for (int j = 0; j < np; j += U) {
                    const double2 q01 = *reinterpret_cast<const double2 *>(lq + j), q23 = *reinterpret_cast<const double2 *>(lq + j + 2);
                    int acc = kIntMax;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double c = c9[IS9 ? r : 0];
                        const int h0 = hi32(fma(x[r], q01.x, c)), h1 = hi32(fma(x[r], q01.y, c));
                        const int h2 = hi32(fma(x[r], q23.x, c)), h3 = hi32(fma(x[r], q23.y, c));
                        acc = min(acc, min(min(h0, h1), min(h2, h3)) - hi32(bt[r]));
                    }
                    if (__any_sync(kFull, acc <= 0)) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            const double c = c9[IS9 ? r : 0];
                            const int h0 = hi32(fma(x[r], q01.x, c)), h1 = hi32(fma(x[r], q01.y, c));
                            const int h2 = hi32(fma(x[r], q23.x, c)), h3 = hi32(fma(x[r], q23.y, c));
                            if (__any_sync(kFull, min(min(h0, h1), min(h2, h3)) <= hi32(bt[r]))) {
#pragma unroll 1
                                for (int u = 0; u < U; ++u) offer(bt[r], bidx[r], fma(x[r], lq[j + u], c), static_cast<uint32_t>(j + u));
                            }
                        }
                    }
                }
                stage(bt, bidx);
            };
            if (q == 0) sweep_q(std::false_type{});
            else if (q == 2) sweep_q(std::true_type{});
            else {
                // ---- id 5: list of (B, C) ----
                const double2 e_pilot = sm.ep[mi];
                const int tc = sm.pc[2 * mi + 1];
                double pm1[R], bt[R];
                uint32_t bidx[R];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    pm1[r] = sm.pm1[32 * r + lane];
                    bt[r] = fma(pm1[r], e_pilot.x, e_pilot.y);
                    bidx[r] = static_cast<uint32_t>(tc);
                }
#pragma unroll 1
                for (int j = 0; j < np; j += U) {
                    const double2 e0 = l5[j], e1 = l5[j + 1], e2 = l5[j + 2], e3 = l5[j + 3];
                    int acc = kIntMax;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const int h0 = hi32(fma(pm1[r], e0.x, e0.y)), h1 = hi32(fma(pm1[r], e1.x, e1.y));
                        const int h2 = hi32(fma(pm1[r], e2.x, e2.y)), h3 = hi32(fma(pm1[r], e3.x, e3.y));
                        acc = min(acc, min(min(h0, h1), min(h2, h3)) - hi32(bt[r]));
                    }
                    if (__any_sync(kFull, acc <= 0)) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            const int h0 = hi32(fma(pm1[r], e0.x, e0.y)), h1 = hi32(fma(pm1[r], e1.x, e1.y));
                            const int h2 = hi32(fma(pm1[r], e2.x, e2.y)), h3 = hi32(fma(pm1[r], e3.x, e3.y));
                            if (__any_sync(kFull, min(min(h0, h1), min(h2, h3)) <= hi32(bt[r]))) {
#pragma unroll 1
                                for (int u = 0; u < U; ++u) {
                                    const double2 e = l5[j + u];
                                    offer(bt[r], bidx[r], fma(pm1[r], e.x, e.y), static_cast<uint32_t>(j + u));
                                }
                            }
                        }
                    }
                }
                stage(bt, bidx);
            }
        }
        __syncthreads();

        // transposed write-out of the strategy's plane: rows of 16 consecutive m per process count
        double *plane_t = p.p_time + (static_cast<size_t>(table - p.out_table0) * 13 + ids[q]) * plane;
        uint32_t *plane_s = p.p_best_s ? p.p_best_s + (static_cast<size_t>(table - p.out_table0) * 3 + q) * plane : nullptr;
        if (p.vec_out) {
            // two message sizes per lane (16-byte and 8-byte stores; the host has checked the alignment), running pointers
            constexpr int kHalf = kSegMG / 2, kRows = 32 / kHalf, kStep = kSegWarps * kRows;
            const int mi = 2 * (lane & (kHalf - 1)), pr0 = warp * kRows + lane / kHalf;
            if (mi < n_mi) {  // n_m is even, so mi + 1 is a message size of the grid too
                const uint32_t m_u0 = p.G.m_list[m0 + mi], m_u1 = p.G.m_list[m0 + mi + 1];
                const size_t cell0 = static_cast<size_t>(tile0 + pr0) * p.G.n_m + static_cast<size_t>(m0 + mi);
                const size_t step = static_cast<size_t>(kStep) * p.G.n_m;
                const double *st0 = sm.st_time + mi * kStride + pr0, *st1 = st0 + kStride;
                const uint16_t *si0 = sm.st_idx + mi * kIStride + pr0, *si1 = si0 + kIStride;
                double *out_t = plane_t + cell0;
                uint32_t *out_s = plane_s ? plane_s + cell0 : nullptr;
                for (int pr = pr0; pr < n_valid; pr += kStep) {
                    *reinterpret_cast<double2 *>(out_t) = make_double2(*st0, *st1);
                    if (out_s) {
                        const uint32_t i0 = *si0, i1 = *si1;
                        *reinterpret_cast<uint2 *>(out_s) = make_uint2(i0 == kWhole ? m_u0 : sm.sval[i0], i1 == kWhole ? m_u1 : sm.sval[i1]);
                        out_s += step;
                    }
                    out_t += step;
                    st0 += kStep; st1 += kStep; si0 += kStep; si1 += kStep;
                }
            }
        } else {
            const int mi = lane & (kSegMG - 1), prow = lane / kSegMG, rows = 32 / kSegMG;
            if (mi < n_mi) {
                const uint32_t m_u = p.G.m_list[m0 + mi];
                const double *st = sm.st_time + mi * kStride;
                const uint16_t *si = sm.st_idx + mi * kIStride;
                for (int pr = warp * rows + prow; pr < n_valid; pr += kSegWarps * rows) {
                    const size_t o = static_cast<size_t>(tile0 + pr) * p.G.n_m + static_cast<size_t>(m0 + mi);
                    plane_t[o] = st[pr];
                    if (plane_s) {
                        const uint32_t idx = si[pr];
                        plane_s[o] = idx == kWhole ? m_u : sm.sval[idx];
                    }
                }
            }
        }
        __syncthreads();  // the staging area is free again
    }
}

size_t segmin_smem_bytes(const TableDev &T, const GridDev &G) { return seg_layout(T.npad, G.n_s, nullptr, nullptr); }

cudaError_t launch_segmin(const SegminParams &p, cudaStream_t st)
{
    const size_t smem = segmin_smem_bytes(p.T, p.G);
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024)
        e = cudaFuncSetAttribute(segmin_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    const long long blocks = static_cast<long long>(p.n_mgroups) * p.n_ptiles * p.n_tables_launch;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    segmin_kernel<<<static_cast<unsigned>(blocks), kSegThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace plogp
