// envelope_kernel: the segment-size search of Section 3.1 without visiting every (P, m, s) cell.
//
// For a fixed message size m every segmented model of Table 1 is a line in x = P-1 (or in floor(log2 P)):
//   id 2: fma(P-1, Q, L)              Q = g(s) k
//   id 9: fma(floor(log2 P), Q, ceil(log2 P) L)
//   id 5: fma(P-1, B, C)              B = g(s) + L, C = g(s) (k-1)
// Ids 2 and 9 have non-negative multipliers, and a rounded fused multiply-add is monotone in Q, so
// their minimum over s is attained by the smallest Q for every P at once: one reduction per m.
// For id 5 the minimum over s is the lower envelope of the lines.  When g does not decrease along the
// candidate sizes (the host only selects this kernel for such tables) two facts hold:
//   * among candidates with the same segment count k the smallest s has the smallest B and C, so
//     only the first candidate of every run of equal k can ever win (its "representative");
//   * the representatives are sorted by slope B, hence the index of the winner does not grow with P:
//     the winners at two process counts bracket the winners at all counts in between.
// The kernel therefore (A) lists the representatives in shared memory, (B) finds the winner at every
// `coarse`-th process count over the whole list and (C) searches, for each process count, only the
// bracket given by its two coarse neighbours (widened by one entry on each side, which absorbs a
// winner that rounding moved across a bracket end).  All comparisons are the exact ones of the
// exhaustive search: (time, s) in lexicographic order.
//
// One CTA per (table, m).  Results go to the scratch layout that the sweep kernel uses, one row per
// message size: [table][strategy slot][m][P] times and candidate indices; fused_kernel reads them.
#include "device_common.cuh"

namespace plogp {

namespace {

constexpr unsigned kFull = 0xffffffffu;

}  // namespace

__global__ void __launch_bounds__(1024) envelope_kernel(const EnvParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int npad = p.T.npad, T = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = T >> 5;
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    double *s_B = s_tab + 3 * npad;                                   // [rep_cap]
    double *s_C = s_B + p.rep_cap;                                    // [rep_cap]
    double *s_redt = s_C + p.rep_cap;                                 // [32]
    uint32_t *s_I = reinterpret_cast<uint32_t *>(s_redt + 32);        // [rep_cap] candidate index of an entry
    uint32_t *s_k = s_I + p.rep_cap;                                  // [T] exchange of k
    int *s_opt = reinterpret_cast<int *>(s_k + T);                    // [max_coarse]
    int *s_cnt = s_opt + p.max_coarse;                                // [32] + [32]

    const int midx = blockIdx.x, trel = blockIdx.y, table = p.table0 + trel;
    const uint32_t m_u = p.G.m_list[midx];
    const int ns = p.G.ns_of_m[midx];
    if (ns == 0) return;  // no candidate fits: the consumer evaluates the whole message itself
    const uint32_t mask = p.G.mask;
    const bool has2 = (mask >> 2) & 1u, has5 = (mask >> 5) & 1u, has9 = (mask >> 9) & 1u;
    const int slot2 = 0, slot5 = has2 ? 1 : 0, slot9 = slot5 + (has5 ? 1 : 0);
    const int n_P = p.G.n_P;
    auto out_row = [&](int slot) { return ((static_cast<size_t>(trel) * p.n_seg + slot) * p.G.n_m + midx) * n_P; };

    stage_table(s_tab, p.T, table);
    __syncthreads();
    const double L = p.T.lat[table];

    // ---- (A) one pass over the candidates: smallest Q, and the representatives of window `win` ----
    double qmin = CUDART_INF;
    int qidx = 0x7FFFFFFF;
    int n_rep = 0;  // all representatives (of every window), known after the first pass
    constexpr int V = 4;  // consecutive candidates per thread and chunk (independent searches and divisions in flight)
    auto list_pass = [&](int win) {
        int base = 0;
        uint32_t carry_k = 0;  // thread 0: k of the last candidate of the previous chunk
        for (int c0 = 0; c0 < ns; c0 += V * T) {
            double gs[V];
            uint32_t k[V];
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int si = c0 + V * tid + v;
                gs[v] = 0.0;
                k[v] = 0;
                if (si < ns) {
                    const uint32_t s = s_at(p.G, si);
                    gs[v] = gap_at(s_tab, npad, static_cast<double>(s));
                    k[v] = segments(m_u, s, p.G.k_mode);
                    if (win == 0) {
                        const double Q = gs[v] * static_cast<double>(k[v]);
                        if (Q < qmin) { qmin = Q; qidx = si; }  // ascending si per thread: the smallest index stays
                    }
                }
            }
            s_k[tid] = k[V - 1];
            __syncthreads();
            uint32_t k_prev = tid > 0 ? s_k[tid - 1] : carry_k;
            unsigned rep = 0;  // bit v: candidate v starts a run of equal segment count
            int cnt = 0;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int si = c0 + V * tid + v;
                if (si < ns && (si == 0 || k[v] != k_prev)) { rep |= 1u << v; ++cnt; }
                k_prev = k[v];
            }
            // ordered positions: inclusive scan of the counts over the warp, then the warps' totals
            int incl = cnt;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int y = __shfl_up_sync(kFull, incl, off);
                if (lane >= off) incl += y;
            }
            if (lane == 31) s_cnt[warp] = incl;
            if (tid == 0) carry_k = s_k[T - 1];
            __syncthreads();
            int off = 0, total = 0;
            for (int w = 0; w < n_warps; ++w) {
                const int c = s_cnt[w];
                off += w < warp ? c : 0;
                total += c;
            }
            int pos = base + off + incl - cnt - win * p.rep_cap;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if ((rep >> v) & 1u) {
                    if (pos >= 0 && pos < p.rep_cap) {
                        s_B[pos] = gs[v] + L;
                        s_C[pos] = gs[v] * (static_cast<double>(k[v]) - 1.0);
                        s_I[pos] = static_cast<uint32_t>(c0 + V * tid + v);
                    }
                    ++pos;
                }
            }
            base += total;
        }
        return base;
    };
    n_rep = list_pass(0);

    // ---- ids 2 and 9: the smallest Q (smallest s on ties) serves every process count ----
    if (has2 || has9) {
        warp_min_pair(qmin, qidx);
        if (lane == 0) { s_redt[warp] = qmin; s_cnt[32 + warp] = qidx; }
        __syncthreads();
        double q = s_redt[0];
        int qi = s_cnt[32];
        for (int w = 1; w < n_warps; ++w) {
            const double q2 = s_redt[w];
            const int i2 = s_cnt[32 + w];
            if (q2 < q || (q2 == q && i2 < qi)) { q = q2; qi = i2; }
        }
        for (int pidx = tid; pidx < n_P; pidx += T) {
            const int P = P_at(p.G, pidx);
            if (has2) {
                p.part_time[out_row(slot2) + pidx] = fma(static_cast<double>(P - 1), q, L);
                p.part_idx[out_row(slot2) + pidx] = static_cast<uint32_t>(qi);
            }
            if (has9) {
                const double lf = static_cast<double>(31 - __clz(P)), lcL = static_cast<double>(32 - __clz(P - 1)) * L;
                p.part_time[out_row(slot9) + pidx] = fma(lf, q, lcL);
                p.part_idx[out_row(slot9) + pidx] = static_cast<uint32_t>(qi);
            }
        }
    }
    if (!has5) return;

    // ---- id 5: lower envelope over the representatives, one window of the list at a time ----
    const int n_c = (n_P - 1 + p.coarse - 1) / p.coarse + 1;  // coarse process-count indices 0, coarse, ..., n_P - 1
    const int n_win = (n_rep + p.rep_cap - 1) / p.rep_cap;
    for (int win = 0; win < n_win; ++win) {
        if (win > 0) {
            __syncthreads();  // the previous window's searches are done with the list
            list_pass(win);
        }
        __syncthreads();
        const int n_e = min(p.rep_cap, n_rep - win * p.rep_cap);
        // (B) winners at the coarse process counts, over the whole window
        for (int c = warp; c < n_c; c += n_warps) {
            const double x = static_cast<double>(P_at(p.G, min(c * p.coarse, n_P - 1)) - 1);
            double tb = CUDART_INF;
            int eb = 0x7FFFFFFF;
            for (int e = lane; e < n_e; e += 32) {
                const double t = fma(x, s_B[e], s_C[e]);
                if (t < tb) { tb = t; eb = e; }
            }
            warp_min_pair(tb, eb);
            if (lane == 0) s_opt[c] = eb;
        }
        __syncthreads();
        // (C) every process count: the bracket of its coarse neighbours, one entry wider on each side
        for (int pidx = tid; pidx < n_P; pidx += T) {
            const int c = pidx / p.coarse;
            const int a = s_opt[min(c + 1, n_c - 1)], b = s_opt[c];
            const int lo = max(min(a, b) - 1, 0), hi = min(max(a, b) + 1, n_e - 1);
            const double x = static_cast<double>(P_at(p.G, pidx) - 1);
            double tb = CUDART_INF;
            int eb = lo;
            for (int e = lo; e <= hi; ++e) {
                const double t = fma(x, s_B[e], s_C[e]);
                if (t < tb) { tb = t; eb = e; }  // ascending e: the smallest s stays on ties
            }
            const size_t o = out_row(slot5) + pidx;
            if (win == 0 || tb < p.part_time[o]) {  // later windows hold larger s: strict '<'
                p.part_time[o] = tb;
                p.part_idx[o] = s_I[eb];
            }
        }
    }
}

size_t envelope_smem_bytes(const TableDev &T, int threads, int rep_cap, int max_coarse)
{
    return (3 * static_cast<size_t>(T.npad) + 2 * static_cast<size_t>(rep_cap) + 32) * sizeof(double) +
           (static_cast<size_t>(rep_cap) + threads) * sizeof(uint32_t) + (static_cast<size_t>(max_coarse) + 64) * sizeof(int);
}

cudaError_t launch_envelope(const EnvParams &p, int threads, cudaStream_t st)
{
    const size_t smem = envelope_smem_bytes(p.T, threads, p.rep_cap, p.max_coarse);
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024)
        e = cudaFuncSetAttribute(envelope_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    if (p.G.n_m <= 0 || p.n_tables_launch <= 0 || p.n_tables_launch > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(p.G.n_m), static_cast<unsigned>(p.n_tables_launch));
    envelope_kernel<<<grid, threads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace plogp
