// CUDA kernels (sm_100a) for the pLogP cost models of Table 1 (Broadcast) and Table 2 (Scatter)
// of "Fast Tuning of Intra-Cluster Collective Communications", the segment-size search of
// Section 3.1 and the strategy selection of Sections 1 and 5.
//
// This file:
//   sweep_kernel   lane <-> process count P.  One CTA owns one message size m, a tile of P values
//                  and a chunk of the candidate segment sizes; the per-(m, s) line coefficients are
//                  computed once per CTA into shared memory and broadcast to all lanes, so a model
//                  cell costs one DFMA and one integer compare.  Used when the candidate list is long.
//   fused_kernel   lane <-> message size m (32 consecutive m per warp, so every output row is
//                  written as full, aligned segments).  Evaluates all enabled strategies, runs short
//                  candidate lists inline or reduces the sweep kernel's partial minima, keeps the
//                  Scatter Chain sum running along each warp's contiguous run of P, and writes either
//                  the predicted planes or the decision table.  The general path.
//   s1_tile_sum    per-tile and per-warp-run sums for the Scatter Chain sum when P is split over CTAs
//                  (reduce-then-scan: the consumers add up the sums of the tiles in front of theirs).
// Short candidate lists have faster, specialised kernels: decide.cu (Broadcast half of the decision
// table), scatter.cu (Scatter half), segmin.cu (segmented planes of the predictions); the host routes
// them there, so fused_kernel's own inline loop over short lists only serves callers of launch_fused
// that pass segmented strategies without partial minima.
#include "device_common.cuh"

namespace plogp {

// ------------------------------------------------------------------------------------------
// Segment sweep: partial minima over one chunk of candidates (Section 3.1 search)
// ------------------------------------------------------------------------------------------
//
// For a fixed (m, s) every segmented model of Table 1 is a line in P (or in floor(log2 P)):
//   id 5: (P-1) (g(s)+L) + g(s)(k-1)          = fma(P-1, B, C)   B = g(s)+L, C = g(s)(k-1)
//   id 2: (P-1) (g(s) k) + L                  = fma(P-1, Q, L)   Q = g(s) k
//   id 9: floor(log2 P) g(s) k + ceil(log2 P) L = fma(lf, Q, lc L)
// so the CTA computes (B, C, Q) once per candidate and every lane spends one DFMA and one
// compare per cell.

template <int SEGMASK>
__global__ void __launch_bounds__(kThreads, 2) sweep_kernel(const SweepParams p)
{
    constexpr bool HAS2 = (SEGMASK & 1) != 0, HAS5 = (SEGMASK & 2) != 0, HAS9 = (SEGMASK & 4) != 0;
    constexpr int R = kSweepR;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    double2 *s_bc = reinterpret_cast<double2 *>(s_tab + 3 * p.T.npad);  // [2][kSweepSub]
    double *s_q = reinterpret_cast<double *>(s_bc + 2 * kSweepSub);     // [2][kSweepSub]

    const int tid = threadIdx.x;
    const int pi = blockIdx.x / p.n_ptiles;
    const int ptile = blockIdx.x - pi * p.n_ptiles;
    const int trel = blockIdx.y;
    const int table = p.table0 + trel;
    const int m_idx = p.pair_m[pi];
    const int chunk = p.pair_chunk[pi];
    const int row = p.pair_row[pi];
    const uint32_t m_u = p.G.m_list[m_idx];
    const int ns = p.G.ns_of_m[m_idx];
    const int s_begin = chunk * p.chunk_len;
    const int s_end = min(ns, s_begin + p.chunk_len);
    const int n_sub = (s_end - s_begin + kSweepSub - 1) / kSweepSub;

    stage_table(s_tab, p.T, table);
    const double L = p.T.lat[table];

    // A warp owns 256 consecutive process counts (lane + 32 r), so neighbouring cells see similar optima
    // and the stores below stay coalesced.
    const int lane = tid & 31, warp = tid >> 5;
    const int p_first = ptile * (kThreads * R) + warp * (32 * R) + lane;
    double pm1[R], best2[R], best5[R], best9[R], lf[R], lcL[R];
    uint32_t idx2[R], idx5[R], idx9[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int pidx = min(p_first + 32 * r, p.G.n_P - 1);
        const int P = P_at(p.G, pidx);
        pm1[r] = static_cast<double>(P - 1);
        lf[r] = static_cast<double>(31 - __clz(P));
        lcL[r] = static_cast<double>(32 - __clz(P - 1)) * L;
        best2[r] = best5[r] = best9[r] = CUDART_INF;
        idx2[r] = idx5[r] = idx9[r] = 0xFFFFFFFFu;
    }
    __syncthreads();

    auto fill = [&](int sub, int buf) {
        const int si = s_begin + sub * kSweepSub + tid;
        double B = CUDART_INF, C = CUDART_INF, Q = CUDART_INF;  // padding never wins a strict '<'
        if (si < s_end) {
            const uint32_t s = s_at(p.G, si);
            const double gs = gap_at(s_tab, p.T.npad, static_cast<double>(s));
            const double k = static_cast<double>(segments(m_u, s, p.G.k_mode));
            B = gs + L;
            C = gs * (k - 1.0);
            Q = gs * k;
        }
        s_bc[buf * kSweepSub + tid] = make_double2(B, C);
        s_q[buf * kSweepSub + tid] = Q;
    };

    fill(0, 0);
    __syncthreads();
    for (int sub = 0; sub < n_sub; ++sub) {
        const int buf = sub & 1;
        if (sub + 1 < n_sub) fill(sub + 1, buf ^ 1);
        const double2 *bc = s_bc + buf * kSweepSub;
        const double *qq = s_q + buf * kSweepSub;
        const uint32_t base = static_cast<uint32_t>(s_begin + sub * kSweepSub);
#pragma unroll 1
        for (int i = 0; i < kSweepSub; i += kSweepU) {
            // Hot path: every cell is evaluated (one DFMA); the comparison with the running minimum is
            // first taken on the high words only, in the integer pipe.  Times are non-negative, so the
            // high word of a smaller double is never larger: a cell can only improve if that test holds.
            // (one flag per register cell: a single flag would chain all the integer compares of the
            // chunk through one predicate, and that dependent chain, not a pipe, then sets the pace)
            bool f5[R], f2[R], f9[R];
#pragma unroll
            for (int r = 0; r < R; ++r) f5[r] = f2[r] = f9[r] = false;
#pragma unroll
            for (int u = 0; u < kSweepU; ++u) {
                if (HAS5) {
                    const double2 c = bc[i + u];
#pragma unroll
                    for (int r = 0; r < R; ++r)
                        f5[r] |= __double2hiint(fma(pm1[r], c.x, c.y)) <= __double2hiint(best5[r]);
                }
                if (HAS2 || HAS9) {
                    const double q = qq[i + u];
                    if (HAS2) {
#pragma unroll
                        for (int r = 0; r < R; ++r)
                            f2[r] |= __double2hiint(fma(pm1[r], q, L)) <= __double2hiint(best2[r]);
                    }
                    if (HAS9) {
#pragma unroll
                        for (int r = 0; r < R; ++r)
                            f9[r] |= __double2hiint(fma(lf[r], q, lcL[r])) <= __double2hiint(best9[r]);
                    }
                }
            }
            bool any5 = false, any2 = false, any9 = false;
#pragma unroll
            for (int r = 0; r < R; r += 2) {
                any5 |= f5[r] | f5[r + 1];
                any2 |= f2[r] | f2[r + 1];
                any9 |= f9[r] | f9[r + 1];
            }
            // Exact passes over the same candidates, in ascending order, strict '<' (smallest s on ties).
            if (HAS5 && any5) {
#pragma unroll 1
                for (int u = 0; u < kSweepU; ++u) {
                    const double2 c = bc[i + u];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double t = fma(pm1[r], c.x, c.y);
                        if (t < best5[r]) { best5[r] = t; idx5[r] = base + i + u; }
                    }
                }
            }
            if (HAS2 && any2) {
#pragma unroll 1
                for (int u = 0; u < kSweepU; ++u) {
                    const double q = qq[i + u];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double t = fma(pm1[r], q, L);
                        if (t < best2[r]) { best2[r] = t; idx2[r] = base + i + u; }
                    }
                }
            }
            if (HAS9 && any9) {
#pragma unroll 1
                for (int u = 0; u < kSweepU; ++u) {
                    const double q = qq[i + u];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double t = fma(lf[r], q, lcL[r]);
                        if (t < best9[r]) { best9[r] = t; idx9[r] = base + i + u; }
                    }
                }
            }
        }
        __syncthreads();
    }

    // partial results, one row per (table, strategy slot, (m, chunk) pair), P contiguous
    int slot = 0;
    auto store = [&](const double *best, const uint32_t *idx) {
        const size_t rbase = (static_cast<size_t>(trel) * p.n_seg + slot) * p.n_pairs + row;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int pidx = p_first + 32 * r;
            if (pidx < p.G.n_P) {
                p.part_time[rbase * p.G.n_P + pidx] = best[r];
                p.part_idx[rbase * p.G.n_P + pidx] = idx[r];
            }
        }
        ++slot;
    };
    if (HAS2) store(best2, idx2);
    if (HAS5) store(best5, idx5);
    if (HAS9) store(best9, idx9);
}

// ------------------------------------------------------------------------------------------
// Scatter Chain: per-tile sums of g(j m) (first phase of the reduce-then-scan over P)
// ------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kThreads) s1_tile_sum_kernel(const S1Params p)
{
    constexpr int R = kFusedR;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    double *s_red = s_tab + 3 * p.T.npad;  // [kWarps][32]

    int b = blockIdx.x;
    const int mtile = b % p.n_mtiles;
    b /= p.n_mtiles;
    const int ptile = b % p.n_ptiles;
    const int trel = b / p.n_ptiles;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int midx = mtile * 32 + lane;
    const double md = static_cast<double>(p.G.m_list[min(midx, p.G.n_m - 1)]);

    stage_table(s_tab, p.T, p.table0 + trel);
    __syncthreads();

    double acc = 0.0;
    GapWalk walk;
    const int run_len = p.passes_per_tile * R;
    const int p_warp = ptile * (kWarps * run_len) + warp * run_len;
    for (int e = 0; e < run_len; ++e)
        if (p_warp + e < p.G.n_P) acc += s1_term(s_tab, p.T.npad, p.G, p_warp + e, md, walk);
    // Per tile and message size: the shares of the 8 warps (each the sum over its run of process counts) and
    // their total, laid out as [tile][9][m]; the kernels that follow turn them into the sum in front of a run.
    s_red[warp * 32 + lane] = acc;
    __syncthreads();
    if (midx < p.G.n_m) {
        double *row = p.tile_sum + (static_cast<size_t>(trel) * p.n_ptiles + ptile) * (kWarps + 1) * p.G.n_m + midx;
        row[static_cast<size_t>(warp) * p.G.n_m] = acc;
        if (warp == 0) {
            double t = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) t += s_red[w * 32 + lane];
            row[static_cast<size_t>(kWarps) * p.G.n_m] = t;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Fused evaluation: all strategies, strategy selection, stores
// ------------------------------------------------------------------------------------------

struct FusedSmem {
    double *tab, *cum, *tot, *gs, *cB, *cC, *cQ;
};

__host__ __device__ inline size_t fused_smem_layout(int npad, int lc_max, int n_inline, FusedSmem *out)
{
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off += n; return o; };
    const size_t o_tab = take(3 * (size_t)npad), o_cum = take((size_t)lc_max * 32),
                 o_tot = take(2 * kWarps * 32), o_gs = take(n_inline), o_B = take((size_t)n_inline * 32),
                 o_C = take((size_t)n_inline * 32), o_Q = take((size_t)n_inline * 32);
    if (out) {
        double *base = out->tab;
        out->tab = base + o_tab; out->cum = base + o_cum; out->tot = base + o_tot; out->gs = base + o_gs;
        out->cB = base + o_B; out->cC = base + o_C; out->cQ = base + o_Q;
    }
    return off * sizeof(double);
}

size_t fused_smem_bytes(const TableDev &T, const GridDev &G, bool inline_sweep)
{
    return fused_smem_layout(T.npad, G.lc_max, inline_sweep ? max(G.n_s, 1) : 1, nullptr);
}

template <bool PREDICT>
__global__ void __launch_bounds__(kThreads, 2) fused_kernel(const FusedParams p)
{
    constexpr int R = kFusedR;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const bool inline_sweep = p.part_time == nullptr;
    const int n_inline = inline_sweep ? max(p.G.n_s, 1) : 1;
    FusedSmem sm;
    sm.tab = reinterpret_cast<double *>(smem_raw);
    fused_smem_layout(p.T.npad, p.G.lc_max, n_inline, &sm);
    const int npad = p.T.npad;
    const uint32_t mask = p.G.mask;
    const bool any_seg = (mask & ((1u << 2) | (1u << 5) | (1u << 9))) != 0;

    int b = blockIdx.x;
    const int mtile = b % p.n_mtiles;
    b /= p.n_mtiles;
    const int ptile = b % p.n_ptiles;
    const int trel = b / p.n_ptiles;
    const int table = p.table0 + trel;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int midx = mtile * 32 + lane;
    const bool m_ok = midx < p.G.n_m;
    const int midx_c = min(midx, p.G.n_m - 1);
    const uint32_t m_u = p.G.m_list[midx_c];
    const double md = static_cast<double>(m_u);
    const int ns = p.G.ns_of_m[midx_c];

    stage_table(sm.tab, p.T, table);
    __syncthreads();

    const double L = p.T.lat[table];
    const double g1 = gap_at(sm.tab, npad, 1.0);
    const double gm = gap_at(sm.tab, npad, md);

    // Scatter Binomial Tree: running sums of g(2^j m), j = 0..lc_max-1 (Table 2, third row)
    // (the gaps are looked up by all warps, one j per warp at a time; warp 0 then adds them up)
    if ((mask >> 12) & 1u) {
        for (int d = warp; d < p.G.lc_max; d += kWarps)
            sm.cum[d * 32 + lane] = gap_at(sm.tab, npad, md * static_cast<double>(1ull << d));
        __syncthreads();
        if (warp == 0) {
            double acc = 0.0;
            for (int d = 0; d < p.G.lc_max; ++d) {
                acc += sm.cum[d * 32 + lane];
                sm.cum[d * 32 + lane] = acc;
            }
        }
    }
    // Inline candidate list: g(s) once per s, then the line coefficients per (s, m)
    if (inline_sweep && any_seg) {
        for (int si = tid; si < p.G.n_s; si += kThreads)
            sm.gs[si] = gap_at(sm.tab, npad, static_cast<double>(s_at(p.G, si)));
        __syncthreads();
        for (int si = warp; si < p.G.n_s; si += kWarps) {
            if (si < ns) {
                const uint32_t s = s_at(p.G, si);
                const double gs = sm.gs[si];
                const double k = static_cast<double>(segments(m_u, s, p.G.k_mode));
                sm.cB[si * 32 + lane] = gs + L;
                sm.cC[si * 32 + lane] = gs * (k - 1.0);
                sm.cQ[si * 32 + lane] = gs * k;
            }
        }
    }
    __syncthreads();

    // Process counts of the tile: warp w owns the contiguous run [w * run_len, (w + 1) * run_len), R of them
    // per pass, so that the Scatter Chain sum can run along a thread without a barrier per pass.
    const int run_len = p.passes_per_tile * R;
    const int p_warp = ptile * (kWarps * run_len) + warp * run_len;

    // Scatter Chain: prefix of g(j m) in front of this thread's run = the tiles in front (sums from
    // s1_tile_sum_kernel when the P range is split over CTAs) + the runs of the lower warps
    double s1_run = 0.0;
    GapWalk s1_walk;  // table interval of this thread's last Scatter Chain argument
    if ((mask >> 11) & 1u) {
        if (p.s1_sums) {
            s1_run = chain_prefix(p.s1_sums, trel, p.n_ptiles, ptile, warp, lane, p.G.n_m, midx_c, sm.tot);
        } else {
            double mine = 0.0;
            for (int e = 0; e < run_len; ++e)
                if (p_warp + e < p.G.n_P) mine += s1_term(sm.tab, npad, p.G, p_warp + e, md, s1_walk);
            sm.tot[warp * 32 + lane] = mine;
            __syncthreads();
            for (int w = 0; w < warp; ++w) s1_run += sm.tot[w * 32 + lane];
            s1_walk.i = -1;
        }
    }

    const size_t plane = static_cast<size_t>(p.G.n_P) * p.G.n_m;

    for (int pass = 0; pass < p.passes_per_tile; ++pass) {
        const int p0 = p_warp + pass * R;
        if (p0 >= p.G.n_P) break;  // this warp's run is exhausted (no barriers below)

        int Pv[R];
        bool ok[R];
        double pm1[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            ok[r] = (p0 + r) < p.G.n_P;
            Pv[r] = P_at(p.G, min(p0 + r, p.G.n_P - 1));
            pm1[r] = static_cast<double>(Pv[r] - 1);
        }

        // ---- Scatter Chain: running sum of g(j m) along the thread's run ----
        double s1sum[R];
        if ((mask >> 11) & 1u) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (ok[r]) s1_run += s1_term(sm.tab, npad, p.G, p0 + r, md, s1_walk);
                s1sum[r] = s1_run;
            }
        }

        // ---- running decision per cell (strict '<' in ascending id keeps the lowest id on ties) ----
        double bt[R];
        uint32_t bsz[R];
        int bid[R];
#pragma unroll
        for (int r = 0; r < R; ++r) { bt[r] = CUDART_INF; bsz[r] = 0; bid[r] = 255; }

        auto out_index = [&](int id_or_coll, int planes, int r) {
            return (static_cast<size_t>(table - p.out_table0) * planes + id_or_coll) * plane +
                   static_cast<size_t>(p0 + r) * p.G.n_m + midx;
        };
        // Predictions: one pointer per row into the table's first plane; a strategy's plane is id * plane further on.
        // Rows past the last process count and lanes past the last message size compute the last valid cell again
        // (their indices are clamped), so they store the same value to the same address: no predicates on the stores.
        unsigned char *row_t[R];
        if (PREDICT) {
            const size_t tab0 = static_cast<size_t>(table - p.out_table0) * 13 * plane + midx_c;
#pragma unroll
            for (int r = 0; r < R; ++r)
                row_t[r] = reinterpret_cast<unsigned char *>(p.p_time + (tab0 + static_cast<size_t>(min(p0 + r, p.G.n_P - 1)) * p.G.n_m));
        }
        const size_t plane_bytes = plane * sizeof(double);
        auto consider = [&](int id, const double *val, const uint32_t *sval) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (PREDICT) {
                    *reinterpret_cast<double *>(row_t[r] + id * plane_bytes) = val[r];
                } else if (val[r] < bt[r]) {
                    bt[r] = val[r];
                    bid[r] = id;
                    bsz[r] = sval ? sval[r] : 0u;
                }
            }
        };
        auto flush = [&](int coll) {
            if constexpr (!PREDICT) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (ok[r] && m_ok) {
                        const size_t o = out_index(coll == 0 ? p.om.plane_bcast : p.om.plane_scat, p.om.planes, r);
                        p.d_strategy[o] = bid[r] < 16 ? p.om.id_of[bid[r]] : static_cast<uint8_t>(bid[r]);
                        p.d_sbytes[o] = bsz[r];
                        p.d_time[o] = bt[r];
                    }
                    bt[r] = CUDART_INF; bsz[r] = 0; bid[r] = 255;
                }
            }
        };

        // Segmented model `id` (slot = its rank among the enabled segmented ids) reduced over
        // the candidates: a[r] * coef1 + c[r] (ids 2, 9) or a[r] * B + C (id 5).
        auto segmented = [&](int id, int seg_rank, int slot, const double *a, const double *c, bool two_coef) {
            double st[R];
            uint32_t si_best[R], sb[R];
#pragma unroll
            for (int r = 0; r < R; ++r) { st[r] = CUDART_INF; si_best[r] = 0; }
            if (ns == 0) {
                // no candidate fits: the message goes whole (s = m, k = 1)
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    st[r] = two_coef ? fma(a[r], gm + L, 0.0) : fma(a[r], gm, c[r]);
                    sb[r] = m_u;
                }
            } else if (inline_sweep) {
                const double *c1 = two_coef ? sm.cB : sm.cQ;
                for (int si = 0; si < ns; ++si) {
                    const double k1 = c1[si * 32 + lane];
                    const double k2 = two_coef ? sm.cC[si * 32 + lane] : 0.0;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const double t = fma(a[r], k1, two_coef ? k2 : c[r]);
                        if (t < st[r]) { st[r] = t; si_best[r] = static_cast<uint32_t>(si); }
                    }
                }
#pragma unroll
                for (int r = 0; r < R; ++r) sb[r] = s_at(p.G, static_cast<int>(si_best[r]));
            } else {
                // partial minima from the sweep kernel, chunks in ascending candidate order
                const int r0 = p.pair_base[midx_c], r1 = p.pair_base[midx_c + 1];
                for (int row = r0; row < r1; ++row) {
                    const size_t rb = ((static_cast<size_t>(trel) * p.n_seg + slot) * p.n_pairs + row) * p.G.n_P;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const int pr = min(p0 + r, p.G.n_P - 1);  // rows past the end repeat the last one
                        const double t = p.part_time[rb + pr];
                        if (t < st[r]) { st[r] = t; si_best[r] = p.part_idx[rb + pr]; }
                    }
                }
#pragma unroll
                for (int r = 0; r < R; ++r) sb[r] = s_at(p.G, static_cast<int>(si_best[r]));
            }
            if (PREDICT && p.p_best_s) {
#pragma unroll
                for (int r = 0; r < R; ++r)
                    if (ok[r] && m_ok) p.p_best_s[out_index(seg_rank, 3, r)] = sb[r];
            }
            consider(id, st, sb);
        };

        double v[R], lf[R], lc[R], lcL[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            lf[r] = static_cast<double>(31 - __clz(Pv[r]));
            lc[r] = static_cast<double>(32 - __clz(Pv[r] - 1));
            lcL[r] = lc[r] * L;
        }
        double Lr[R];
#pragma unroll
        for (int r = 0; r < R; ++r) Lr[r] = L;
        const double rdv = 2.0 * g1 + 3.0 * L;  // rendezvous handshake: 2 g(1) + 3 L
        int slot = 0;

        // ---- Broadcast, Table 1 ----
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
        if ((mask >> 2) & 1u) segmented(2, 0, slot++, pm1, Lr, false);  // Segmented Flat Tree
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
        if ((mask >> 5) & 1u) segmented(5, 1, slot++, pm1, nullptr, true);  // Segmented Chain
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
        if ((mask >> 9) & 1u) segmented(9, 2, slot++, lf, lcL, false);  // Segmented Binomial Tree
        if (mask & 0x3FFu) flush(0);

        // ---- Scatter, Table 2 ----
        if ((mask >> 10) & 1u) {  // Flat Tree
#pragma unroll
            for (int r = 0; r < R; ++r) v[r] = fma(pm1[r], gm, L);
            consider(10, v, nullptr);
        }
        if ((mask >> 11) & 1u) {  // Chain
#pragma unroll
            for (int r = 0; r < R; ++r) v[r] = fma(pm1[r], L, s1sum[r]);
            consider(11, v, nullptr);
        }
        if ((mask >> 12) & 1u) {  // Binomial Tree
#pragma unroll
            for (int r = 0; r < R; ++r) v[r] = sm.cum[(32 - __clz(Pv[r] - 1) - 1) * 32 + lane] + lcL[r];
            consider(12, v, nullptr);
        }
        if (mask & 0x1C00u) flush(1);
    }
}

// ------------------------------------------------------------------------------------------
// FP64 issue-rate probe (measurement aid)
// ------------------------------------------------------------------------------------------

// 16 independent chains per thread: with fewer, the loop's own counter and branch take issue slots from
// the DFMAs (8 chains reach 0.92 of the 64-lanes-per-SM rate, 12 or more reach 0.997).
constexpr int kProbeChains = 16;
__global__ void __launch_bounds__(kThreads) fp64_probe_kernel(double *sink, int iters)
{
    double a[kProbeChains];
    const double x = 1.0 + 1e-9 * threadIdx.x, y = 1e-12 * blockIdx.x;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) a[i] = 0.5 + i;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
#pragma unroll
            for (int i = 0; i < kProbeChains; ++i) a[i] = fma(a[i], x, y);
        }
    }
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) s += a[i];
    if (s == 1234.5678) sink[0] = s;  // keeps the chains alive; practically never true
}

// ------------------------------------------------------------------------------------------
// Launch wrappers
// ------------------------------------------------------------------------------------------

template <typename K>
static cudaError_t set_smem(K kernel, size_t bytes)
{
    if (bytes <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
}

cudaError_t launch_fused(const FusedParams &p, bool predict, cudaStream_t st)
{
    const size_t smem = fused_smem_bytes(p.T, p.G, p.part_time == nullptr);
    const long long blocks = static_cast<long long>(p.n_mtiles) * p.n_ptiles * p.n_tables_launch;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    cudaError_t e;
    if (predict) {
        if ((e = set_smem(fused_kernel<true>, smem)) != cudaSuccess) return e;
        fused_kernel<true><<<static_cast<unsigned>(blocks), kThreads, smem, st>>>(p);
    } else {
        if ((e = set_smem(fused_kernel<false>, smem)) != cudaSuccess) return e;
        fused_kernel<false><<<static_cast<unsigned>(blocks), kThreads, smem, st>>>(p);
    }
    return cudaGetLastError();
}

template <int SEGMASK>
static cudaError_t launch_sweep_t(const SweepParams &p, int n_tables_launch, cudaStream_t st)
{
    const size_t smem = 3 * static_cast<size_t>(p.T.npad) * sizeof(double) +
                        2 * kSweepSub * (sizeof(double2) + sizeof(double));
    cudaError_t e = set_smem(sweep_kernel<SEGMASK>, smem);
    if (e != cudaSuccess) return e;
    const long long bx = static_cast<long long>(p.n_pairs) * p.n_ptiles;
    if (bx <= 0 || bx > 0x7FFFFFFFLL || n_tables_launch > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(bx), static_cast<unsigned>(n_tables_launch));
    sweep_kernel<SEGMASK><<<grid, kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_sweep(const SweepParams &p, int n_tables_launch, cudaStream_t st)
{
    const uint32_t m = p.G.mask;
    const int segmask = ((m >> 2) & 1) | (((m >> 5) & 1) << 1) | (((m >> 9) & 1) << 2);
    switch (segmask) {
    case 1: return launch_sweep_t<1>(p, n_tables_launch, st);
    case 2: return launch_sweep_t<2>(p, n_tables_launch, st);
    case 3: return launch_sweep_t<3>(p, n_tables_launch, st);
    case 4: return launch_sweep_t<4>(p, n_tables_launch, st);
    case 5: return launch_sweep_t<5>(p, n_tables_launch, st);
    case 6: return launch_sweep_t<6>(p, n_tables_launch, st);
    case 7: return launch_sweep_t<7>(p, n_tables_launch, st);
    default: return cudaSuccess;
    }
}

cudaError_t launch_s1_tiles(const S1Params &p, cudaStream_t st)
{
    const size_t smem = (3 * static_cast<size_t>(p.T.npad) + kWarps * 32) * sizeof(double);
    cudaError_t e = set_smem(s1_tile_sum_kernel, smem);
    if (e != cudaSuccess) return e;
    const long long blocks = static_cast<long long>(p.n_mtiles) * p.n_ptiles * p.n_tables_launch;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    s1_tile_sum_kernel<<<static_cast<unsigned>(blocks), kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_fp64_probe(double *d_sink, int iters, int blocks, cudaStream_t st)
{
    fp64_probe_kernel<<<blocks, kThreads, 0, st>>>(d_sink, iters);
    return cudaGetLastError();
}

}  // namespace plogp
