// decide_kernel: Broadcast half of the decision table (Sections 1 and 5 of the paper) for short
// candidate lists, with lanes mapped to the process count P.  (The Scatter half has no candidate
// lists and goes through scatter_kernel.)
//
// One CTA owns one table, a group of 8 message sizes and a tile of 512 process counts (4 warps x
// 32 lanes x 4 cells).  For a fixed (m, s) the segmented models of Table 1 are lines in P, so the
// CTA computes the line coefficients once per (m, s) into shared memory and every lane reads them
// with one broadcast load.  Each model cell is evaluated with one DFMA.  The comparison with the
// running minimum is first made on the high 32 bits in the integer pipe (times are non-negative,
// so a smaller double never has a larger high word); only chunks of candidates in which some cell
// can improve run the exact FP64 compare-and-select pass.  To make that pass rare, each warp first
// finds the best candidate for the process count in the middle of its range (one candidate per
// lane, one warp-wide integer minimum over float keys) and evaluates that candidate's chunk first: neighbouring process counts
// nearly always share the optimum, and for ids 2 and 9 the optimum does not depend on P at all.
//
// Results are staged in shared memory as [m][P] and written out as rows of 8 consecutive m.
#include "device_common.cuh"

#include <algorithm>

namespace plogp {

namespace {

constexpr int kDecStride = kDecTileP + 2;  // doubles per staged row: keeps the transposed reads conflict-free

struct DecSmem {
    double *tab, *gs, *cQ, *gm, *st_time;
    double2 *cBC;
    uint8_t *st_id, *st_si;
};

__host__ __device__ inline size_t dec_layout(int npad, int nsp, unsigned char *base, DecSmem *o)
{
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += (bytes + 15) & ~size_t(15); return at; };
    const size_t o_tab = take(3 * size_t(npad) * 8), o_gs = take(size_t(nsp) * 8), o_BC = take(size_t(kDecMG) * nsp * 16),
                 o_Q = take(size_t(kDecMG) * nsp * 8), o_gm = take(kDecMG * 8), o_t = take(size_t(kDecMG) * kDecStride * 8),
                 o_id = take(size_t(kDecMG) * (kDecTileP + 16)), o_si = take(size_t(kDecMG) * (kDecTileP + 16));
    if (o) {
        o->tab = reinterpret_cast<double *>(base + o_tab); o->gs = reinterpret_cast<double *>(base + o_gs);
        o->cBC = reinterpret_cast<double2 *>(base + o_BC); o->cQ = reinterpret_cast<double *>(base + o_Q);
        o->gm = reinterpret_cast<double *>(base + o_gm); o->st_time = reinterpret_cast<double *>(base + o_t);
        o->st_id = base + o_id; o->st_si = base + o_si;
    }
    return off;
}

constexpr uint8_t kSiNone = 255;      // winner is an unsegmented strategy
constexpr uint8_t kSiWhole = 254;     // segmented winner with no fitting candidate: the whole message


}  // namespace

__global__ void __launch_bounds__(kDecThreads, 4) decide_kernel(const DecideParams p)
{
    constexpr int R = kDecR, U = kDecU;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int npad = p.T.npad;
    const int nsp = (max(p.G.n_s, 1) + U - 1) / U * U;
    DecSmem sm;
    dec_layout(npad, nsp, smem_raw, &sm);
    const uint32_t mask = p.G.mask;

    int b = blockIdx.x;
    const int mgroup = b % p.n_mgroups;
    b /= p.n_mgroups;
    const int ptile = b % p.n_ptiles;
    const int trel = b / p.n_ptiles;
    const int table = p.table0 + trel;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = mgroup * p.mg;   // p.mg <= kDecMG message sizes per CTA (fewer on small grids, for more CTAs)
    const int n_mi = min(p.mg, p.G.n_m - m0);

    stage_table(sm.tab, p.T, table);
    __syncthreads();
    const double L = p.T.lat[table];
    for (int si = tid; si < p.G.n_s; si += kDecThreads)
        sm.gs[si] = gap_at(sm.tab, npad, static_cast<double>(s_at(p.G, si)));
    if (tid >= kDecThreads - kDecMG) {  // g(m) of the group's message sizes, by the last threads
        const int mi = tid - (kDecThreads - kDecMG);
        if (mi < n_mi) sm.gm[mi] = gap_at(sm.tab, npad, static_cast<double>(p.G.m_list[m0 + mi]));
    }
    const double g1 = gap_at(sm.tab, npad, 1.0);
    const double rdv = 2.0 * g1 + 3.0 * L;  // rendezvous handshake: 2 g(1) + 3 L
    __syncthreads();
    // line coefficients per (message size of the group, candidate): Section 2's k, Table 1's segmented rows
    for (int idx = tid; idx < n_mi * nsp; idx += kDecThreads) {
        const int mi = idx / nsp, si = idx - mi * nsp;
        const uint32_t m_u = p.G.m_list[m0 + mi];
        const int ns = p.G.ns_of_m[m0 + mi];
        double B = CUDART_INF, C = CUDART_INF, Q = CUDART_INF;  // padding never wins
        if (si < ns) {
            const double gs = sm.gs[si];
            const double k = static_cast<double>(segments(m_u, s_at(p.G, si), p.G.k_mode));
            B = gs + L; C = gs * (k - 1.0); Q = gs * k;
        } else if (ns == 0 && si == 0) {  // nothing fits: the whole message, k = 1
            B = sm.gm[mi] + L; C = 0.0; Q = sm.gm[mi];
        }
        sm.cBC[idx] = make_double2(B, C);
        sm.cQ[idx] = Q;
    }
    __syncthreads();

    // this thread's cells: process counts at tile offset warp*128 + r*32 + lane
    const int p_first = ptile * kDecTileP + warp * (32 * R) + lane;
    int Pv[R];
    double pm1[R], lf[R], lc[R], lcL[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int pidx = p_first + 32 * r;
        Pv[r] = P_at(p.G, min(pidx, p.G.n_P - 1));
        pm1[r] = static_cast<double>(Pv[r] - 1);
        lf[r] = static_cast<double>(31 - __clz(Pv[r]));
        lc[r] = static_cast<double>(32 - __clz(Pv[r] - 1));
        lcL[r] = lc[r] * L;
    }
    // the warp's pilot process count (middle of its range, clamped to the grid)
    const int P_mid = P_at(p.G, min(ptile * kDecTileP + warp * (32 * R) + 16 * R, p.G.n_P - 1));
    const double pm1_mid = static_cast<double>(P_mid - 1);

    // Pilots for the whole group, issued together so that their latencies overlap: for each message size
    // the chunk holding the candidate that is best at the warp's middle process count.  Only a guess that
    // orders the work (float precision, candidate index in the low bits of the key); 4 bits per message size.
    uint32_t pilotQ = 0, pilot5 = 0;
    if (mask & ((1u << 2) | (1u << 5) | (1u << 9))) {
#pragma unroll
        for (int mi = 0; mi < kDecMG; ++mi) {
            if (mi < n_mi) {
                const int nsv = max(p.G.ns_of_m[m0 + mi], 1);
                unsigned kq = 0xFFFFFFFFu, k5 = 0xFFFFFFFFu;
                for (int c0 = 0; c0 < nsv; c0 += 32) {
                    const int cand = c0 + lane;
                    if (cand < nsv) {
                        const double2 c = sm.cBC[mi * nsp + cand];
                        kq = min(kq, (__float_as_uint(static_cast<float>(sm.cQ[mi * nsp + cand])) & ~63u) | static_cast<unsigned>(cand));
                        k5 = min(k5, (__float_as_uint(static_cast<float>(fma(pm1_mid, c.x, c.y))) & ~63u) | static_cast<unsigned>(cand));
                    }
                }
                pilotQ |= ((__reduce_min_sync(0xffffffffu, kq) & 63u) / U) << (4 * mi);
                pilot5 |= ((__reduce_min_sync(0xffffffffu, k5) & 63u) / U) << (4 * mi);
            }
        }
    }

    const size_t plane = static_cast<size_t>(p.G.n_P) * p.G.n_m;

    // transposed write-out of the staged group: rows of n_mi consecutive m per process count
    auto write_out = [&](int coll) {
        const int mi = lane & 7, prow = lane >> 3;
        if (mi < n_mi) {
            const uint32_t m_u = p.G.m_list[m0 + mi];
            for (int pr = warp * 4 + prow; pr < kDecTileP; pr += kDecWarps * 4) {
                const int pidx = ptile * kDecTileP + pr;
                if (pidx >= p.G.n_P) break;
                const size_t o = (static_cast<size_t>(table) * 2 + coll) * plane + static_cast<size_t>(pidx) * p.G.n_m + m0 + mi;
                const uint8_t si = sm.st_si[mi * (kDecTileP + 16) + pr];
                p.d_time[o] = sm.st_time[mi * kDecStride + pr];
                p.d_strategy[o] = sm.st_id[mi * (kDecTileP + 16) + pr];
                p.d_sbytes[o] = si == kSiNone ? 0u : (si == kSiWhole ? m_u : s_at(p.G, si));
            }
        }
    };

    // =============================== Broadcast (Table 1) ===============================
    if (mask & 0x3FFu) {
        for (int mi = 0; mi < n_mi; ++mi) {
            const int midx = m0 + mi;
            const int ns = p.G.ns_of_m[midx];
            const int nsv = max(ns, 1);                 // candidates actually evaluated
            const int n_chunks = (nsv + U - 1) / U;

            const double gm = sm.gm[mi];
            const double2 *cBC = sm.cBC + mi * nsp;
            const double *cQ = sm.cQ + mi * nsp;

            double bt[R];
            uint32_t bcode[R];  // winner so far: strategy id << 8 | candidate index (or kSiNone / kSiWhole)
#pragma unroll
            for (int r = 0; r < R; ++r) { bt[r] = CUDART_INF; bcode[r] = (255u << 8) | kSiNone; }
            auto consider = [&](int id, const double *val, const uint32_t *sval) {
#pragma unroll
                for (int r = 0; r < R; ++r)
                    if (val[r] < bt[r]) { bt[r] = val[r]; bcode[r] = (static_cast<uint32_t>(id) << 8) | (sval ? sval[r] : kSiNone); }
            };

            // Segmented model reduced over the candidates: load(cand) fetches the candidate's line
            // coefficients from shared memory, eval(r, coef) is the model cell.
            auto segmented = [&](int id, int cp, auto load, auto eval) {
                double st[R];
                uint32_t si[R];
#pragma unroll
                for (int r = 0; r < R; ++r) { st[r] = CUDART_INF; si[r] = 0; }
                // the pilot's chunk first, ascending, strict '<'
#pragma unroll 1
                for (int u = 0; u < U; ++u) {
                    const uint32_t cand = cp * U + u;
                    const auto k = load(cand);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double t = eval(r, k);
                        if (t < st[r]) { st[r] = t; si[r] = cand; }
                    }
                }
                // all other chunks; the next chunk's coefficients are fetched before the current one is tested
                decltype(load(0)) cur[U], nxt[U];
                int chunk = cp == 0 ? 1 : 0;
#pragma unroll
                for (int u = 0; u < U; ++u) cur[u] = load(min(chunk, n_chunks - 1) * U + u);
                while (chunk < n_chunks) {
                    int next = chunk + 1;
                    next += next == cp;
#pragma unroll
                    for (int u = 0; u < U; ++u) nxt[u] = load(min(next, n_chunks - 1) * U + u);
                    // one flag per cell: a single flag would chain all 16 integer compares through one predicate
                    bool f[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) f[r] = false;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
#pragma unroll
                        for (int r = 0; r < R; ++r)
                            f[r] |= __double2hiint(eval(r, cur[u])) <= __double2hiint(st[r]);
                    }
                    if ((f[0] | f[1]) | (f[2] | f[3])) {  // exact pass; chunks arrive out of order: ties go to the smaller index
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            const uint32_t cand = chunk * U + u;
#pragma unroll
                            for (int r = 0; r < R; ++r) {
                                const double t = eval(r, cur[u]);
                                if (t < st[r] || (t == st[r] && cand < si[r])) { st[r] = t; si[r] = cand; }
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) cur[u] = nxt[u];
                    chunk = next;
                }
                if (ns == 0) {
#pragma unroll
                    for (int r = 0; r < R; ++r) si[r] = kSiWhole;
                }
                consider(id, st, si);
            };
            // Ids 2 and 9 together: both read Q(s), so one sweep loads it once and tests 32 cells per branch.
            double st9[R];
            uint32_t si9[R];
            auto segmented_2_and_9 = [&](int cp) {
                double st2[R];
                uint32_t si2[R];
#pragma unroll
                for (int r = 0; r < R; ++r) { st2[r] = st9[r] = CUDART_INF; si2[r] = si9[r] = 0; }
#pragma unroll 1
                for (int u = 0; u < U; ++u) {  // the pilot's chunk first, ascending, strict '<'
                    const uint32_t cand = cp * U + u;
                    const double q = cQ[cand];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double t2 = fma(pm1[r], q, L), t9 = fma(lf[r], q, lcL[r]);
                        if (t2 < st2[r]) { st2[r] = t2; si2[r] = cand; }
                        if (t9 < st9[r]) { st9[r] = t9; si9[r] = cand; }
                    }
                }
                double cur[U], nxt[U];
                int chunk = cp == 0 ? 1 : 0;
#pragma unroll
                for (int u = 0; u < U; ++u) cur[u] = cQ[min(chunk, n_chunks - 1) * U + u];
                while (chunk < n_chunks) {
                    int next = chunk + 1;
                    next += next == cp;
#pragma unroll
                    for (int u = 0; u < U; ++u) nxt[u] = cQ[min(next, n_chunks - 1) * U + u];
                    bool f2[R], f9[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) f2[r] = f9[r] = false;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            f2[r] |= __double2hiint(fma(pm1[r], cur[u], L)) <= __double2hiint(st2[r]);
                            f9[r] |= __double2hiint(fma(lf[r], cur[u], lcL[r])) <= __double2hiint(st9[r]);
                        }
                    }
                    const bool a2 = (f2[0] | f2[1]) | (f2[2] | f2[3]), a9 = (f9[0] | f9[1]) | (f9[2] | f9[3]);
                    if (a2 | a9) {  // exact pass (rare); chunks arrive out of order: ties go to the smaller index
#pragma unroll 1
                        for (int u = 0; u < U; ++u) {
                            const uint32_t cand = chunk * U + u;
                            const double q = cQ[cand];
#pragma unroll
                            for (int r = 0; r < R; ++r) {
                                const double t2 = fma(pm1[r], q, L), t9 = fma(lf[r], q, lcL[r]);
                                if (t2 < st2[r] || (t2 == st2[r] && cand < si2[r])) { st2[r] = t2; si2[r] = cand; }
                                if (t9 < st9[r] || (t9 == st9[r] && cand < si9[r])) { st9[r] = t9; si9[r] = cand; }
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) cur[u] = nxt[u];
                    chunk = next;
                }
                if (ns == 0) {
#pragma unroll
                    for (int r = 0; r < R; ++r) si2[r] = si9[r] = kSiWhole;
                }
                consider(2, st2, si2);
            };
            // ids 2 and 9 are a_P * Q(s) + c_P with a_P > 0: their best candidate is the same for every P
            const int cpQ = (pilotQ >> (4 * mi)) & 15;

            double v[R];
            if (mask & 1u) {  // Flat Tree
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = fma(pm1[r], gm, L);
                consider(0, v, nullptr);
            }
            if ((mask >> 1) & 1u) {  // Flat Tree Rendezvous
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = fma(pm1[r], gm, rdv);
                consider(1, v, nullptr);
            }
            const bool both29 = ((mask >> 2) & 1u) && ((mask >> 9) & 1u);
            if (both29) segmented_2_and_9(cpQ);
            else if ((mask >> 2) & 1u)  // Segmented Flat Tree
                segmented(2, cpQ, [&](int cand) { return cQ[cand]; }, [&](int r, double q) { return fma(pm1[r], q, L); });
            if ((mask >> 3) & 1u) {  // Chain
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = pm1[r] * (gm + L);
                consider(3, v, nullptr);
            }
            if ((mask >> 4) & 1u) {  // Chain Rendezvous
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = pm1[r] * (gm + rdv);
                consider(4, v, nullptr);
            }
            if ((mask >> 5) & 1u) {  // Segmented Chain
                const int cp5 = (pilot5 >> (4 * mi)) & 15;
                segmented(5, cp5, [&](int cand) { return cBC[cand]; }, [&](int r, double2 c) { return fma(pm1[r], c.x, c.y); });
            }
            if ((mask >> 6) & 1u) {  // Binary Tree (the printed bound)
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = lc[r] * fma(2.0, gm, L);
                consider(6, v, nullptr);
            }
            if ((mask >> 7) & 1u) {  // Binomial Tree
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = fma(lf[r], gm, lcL[r]);
                consider(7, v, nullptr);
            }
            if ((mask >> 8) & 1u) {  // Binomial Tree Rendezvous
#pragma unroll
                for (int r = 0; r < R; ++r) v[r] = fma(lf[r], gm, lc[r] * rdv);
                consider(8, v, nullptr);
            }
            if (both29) consider(9, st9, si9);
            else if ((mask >> 9) & 1u)  // Segmented Binomial Tree
                segmented(9, cpQ, [&](int cand) { return cQ[cand]; }, [&](int r, double q) { return fma(lf[r], q, lcL[r]); });

#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int pr = warp * (32 * R) + 32 * r + lane;
                sm.st_time[mi * kDecStride + pr] = bt[r];
                sm.st_id[mi * (kDecTileP + 16) + pr] = static_cast<uint8_t>(bcode[r] >> 8);
                sm.st_si[mi * (kDecTileP + 16) + pr] = static_cast<uint8_t>(bcode[r] & 255u);
            }
        }
        __syncthreads();
        write_out(0);
    }
}

size_t decide_smem_bytes(const TableDev &T, const GridDev &G)
{
    const int nsp = (std::max(G.n_s, 1) + kDecU - 1) / kDecU * kDecU;
    return dec_layout(T.npad, nsp, nullptr, nullptr);
}

cudaError_t launch_decide(const DecideParams &p, cudaStream_t st)
{
    const size_t smem = decide_smem_bytes(p.T, p.G);
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024)
        e = cudaFuncSetAttribute(decide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    const long long blocks = static_cast<long long>(p.n_mgroups) * p.n_ptiles * p.n_tables_launch;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    decide_kernel<<<static_cast<unsigned>(blocks), kDecThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace plogp
