// scatter_kernel: Scatter half of the decision table (Table 2 of the paper: Flat Tree, Chain,
// Binomial Tree; selection as in Sections 1 and 5).
//
// Lanes are message sizes (32 consecutive m per warp, so every store is one aligned row segment);
// each warp owns a contiguous run of process counts and walks it in ascending order, which turns
// the Chain model's sum over j = 1..P-1 of g(j m) into a running sum along the thread: the argument
// j m grows by m per step, the table interval is kept in registers and only reloaded when the
// argument crosses a breakpoint.  The sum in front of a warp's run comes from the runs of the lower
// warps (one pass over the run without stores, one barrier) or, when the P range is split over
// several CTAs, from the per-run and per-tile sums that s1_tile_sum_kernel has written (reduce-then-scan).
#include "device_common.cuh"

namespace plogp {

namespace {

// Interval walk without the clamp of gap_at: below the table a pseudo-interval with slope 0
// holds g at its first value.
struct LineWalk {
    int i;
    double key, next, slope, gap;

    __device__ __forceinline__ void start(const double *s_tab, int npad, double x)
    {
        if (x < s_tab[0]) {
            i = -1; key = 0.0; next = s_tab[0]; slope = 0.0; gap = s_tab[npad];
        } else {
            i = interval_of(s_tab, npad, x);
            load(s_tab, npad);
        }
    }
    __device__ __forceinline__ void load(const double *s_tab, int npad)
    {
        key = s_tab[i]; next = s_tab[i + 1]; slope = s_tab[2 * npad + i]; gap = s_tab[npad + i];
    }
    __device__ __forceinline__ double at(const double *s_tab, int npad, double x)
    {
        while (x >= next) {
            // rare: keep it a branch (the barrier stops the compiler from turning the reload into
            // loads and selects that would run at every step)
            asm volatile("" ::: "memory");
            ++i;
            load(s_tab, npad);
        }
        return fma(x - key, slope, gap);
    }
};

}  // namespace

// CONTIG: the process counts are the contiguous range P_lo + index (one new gap per step).
// ALL: the three Scatter strategies are enabled (the usual case), known at compile time.
template <bool CONTIG, bool ALL>
__global__ void __launch_bounds__(kThreads, 4) scatter_kernel(const FusedParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    double *s_cum = s_tab + 3 * p.T.npad;      // [lc_max][32]
    double *s_tot = s_cum + p.G.lc_max * 32;   // [kWarps][32]
    const int npad = p.T.npad;
    const uint32_t mask = p.G.mask;
    const bool on10 = ALL || ((mask >> 10) & 1u), on11 = ALL || ((mask >> 11) & 1u), on12 = ALL || ((mask >> 12) & 1u);

    int b = blockIdx.x;
    const int mtile = b % p.n_mtiles;
    b /= p.n_mtiles;
    const int ptile = b % p.n_ptiles;
    const int trel = b / p.n_ptiles;
    const int table = p.table0 + trel;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int midx = mtile * 32 + lane;
    const bool m_ok = midx < p.G.n_m;
    const int midx_c = min(midx, p.G.n_m - 1);
    const double md = static_cast<double>(p.G.m_list[midx_c]);

    stage_table(s_tab, p.T, table);
    __syncthreads();
    const double L = p.T.lat[table];
    const double gm = gap_at(s_tab, npad, md);

    // Binomial Tree: sums of g(2^j m); the gaps are looked up by all warps, warp 0 adds them up
    if (on12) {
        for (int d = warp; d < p.G.lc_max; d += kWarps)
            s_cum[d * 32 + lane] = gap_at(s_tab, npad, md * static_cast<double>(1ull << d));
        __syncthreads();
        if (warp == 0) {
            double acc = 0.0;
            for (int d = 0; d < p.G.lc_max; ++d) {
                acc += s_cum[d * 32 + lane];
                s_cum[d * 32 + lane] = acc;
            }
        }
    }

    // this warp's run of process-count indices
    const int run_len = p.passes_per_tile * kFusedR;
    const int e0 = ptile * (kWarps * run_len) + warp * run_len;
    const int e1 = min(e0 + run_len, p.G.n_P);

    // Chain sum.  Contiguous process counts: the step for index e is the single gap g((P-1) m), and the
    // argument grows by m per step; only the very first index of the grid also owns the gaps below it
    // (j = 1 .. P_lo - 2).  Listed process counts: the step owns all j from the previous count to P-1.
    auto below_first = [&]() {  // CONTIG, e0 == 0: sum of g(j m), j = 1 .. P_lo - 2 (closed form per table interval)
        return p.G.P_lo > 2 ? chain_range_sum(s_tab, npad, md, 1, p.G.P_lo - 2) : 0.0;
    };
    auto listed_step = [&](int e, int P, LineWalk &w) {  // !CONTIG: all j from the previous listed count to P - 1
        const int jlo = e == 0 ? 1 : P_at(p.G, e - 1);
        if (jlo == P - 1) return w.at(s_tab, npad, static_cast<double>(jlo) * md);
        return chain_range_sum(s_tab, npad, md, jlo, P - 1);
    };
    const int P0 = e0 < p.G.n_P ? P_at(p.G, e0) : 2;
    const double x_first = static_cast<double>((e0 == 0 || !CONTIG) ? (e0 == 0 ? 1 : P_at(p.G, e0 - 1)) : P0 - 1) * md;

    double run = 0.0;
    if (on11 && p.s1_sums) {
        // P range split over CTAs: the sums of the tiles and warp runs in front come from s1_tile_sum_kernel
        run = chain_prefix(p.s1_sums, trel, p.n_ptiles, ptile, warp, lane, p.G.n_m, midx_c, s_tot);  // one barrier inside
    } else {
        if (on11) {  // first pass over the run, no stores: this warp's share of the sum
            double mine = 0.0;
            if (e0 < e1) {
                LineWalk w;
                w.start(s_tab, npad, x_first);
                if (CONTIG) {
                    if (e0 == 0) mine = below_first();
                    double x = static_cast<double>(P0 - 1) * md;
                    for (int e = e0; e < e1; ++e) {
                        mine += w.at(s_tab, npad, x);
                        x += md;  // exact: j m < 2^53
                    }
                } else {
                    for (int e = e0; e < e1; ++e) mine += listed_step(e, P_at(p.G, e), w);
                }
            }
            s_tot[warp * 32 + lane] = mine;
        }
        __syncthreads();  // also publishes s_cum
        if (on11)
            for (int w = 0; w < warp; ++w) run += s_tot[w * 32 + lane];
    }
    if (e0 >= e1 || !m_ok) return;  // no barriers below

    LineWalk w;
    if (on11) {
        w.start(s_tab, npad, x_first);
        if (CONTIG && e0 == 0) run += below_first();
    }
    double x = static_cast<double>(P0 - 1) * md;

    const size_t plane = static_cast<size_t>(p.G.n_P) * p.G.n_m;
    const size_t o = (static_cast<size_t>(table - p.out_table0) * p.om.planes + p.om.plane_scat) * plane + static_cast<size_t>(e0) * p.G.n_m + midx;
    // running output pointers (one row of n_m cells further per process count) and the ids as the caller names them
    double *out_t = p.d_time + o;
    uint8_t *out_id = p.d_strategy + o;
    uint32_t *out_s = p.d_sbytes + o;
    const size_t row = static_cast<size_t>(p.G.n_m);
    const uint8_t id10 = p.om.id_of[10], id11 = p.om.id_of[11], id12 = p.om.id_of[12];
    int P = P0;
    int lc = 32 - __clz(P - 1);               // ceil(log2 P)
    int P_next_lc = (1 << lc) + 1;            // first process count with a larger ceil(log2 P)
    double lcL = static_cast<double>(lc) * L;
    double s2 = on12 ? s_cum[(lc - 1) * 32 + lane] + lcL : 0.0;
    double pm1 = static_cast<double>(P - 1);

    for (int e = e0; e < e1; ++e) {
        if (!CONTIG) {
            P = P_at(p.G, e);
            pm1 = static_cast<double>(P - 1);
        }
        if (P >= P_next_lc) {  // P passed a power of two
            lc = 32 - __clz(P - 1);
            P_next_lc = (1 << lc) + 1;
            lcL = static_cast<double>(lc) * L;
            if (on12) s2 = s_cum[(lc - 1) * 32 + lane] + lcL;
        }
        double bt = CUDART_INF;
        uint8_t bid = 255;
        if (on10) { bt = fma(pm1, gm, L); bid = id10; }                  // Flat Tree
        if (on11) {                                                      // Chain
            if (CONTIG) {
                run += w.at(s_tab, npad, x);
                x += md;
            } else {
                run += listed_step(e, P, w);
            }
            const double t = fma(pm1, L, run);
            if (t < bt) { bt = t; bid = id11; }
        }
        if (on12 && s2 < bt) { bt = s2; bid = id12; }                    // Binomial Tree
        *out_t = bt;
        *out_id = bid;
        *out_s = 0u;
        out_t += row; out_id += row; out_s += row;
        if (CONTIG) { ++P; pm1 += 1.0; }
    }
}

template <bool CONTIG, bool ALL>
static cudaError_t launch_scatter_t(const FusedParams &p, size_t smem, unsigned blocks, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(scatter_kernel<CONTIG, ALL>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    scatter_kernel<CONTIG, ALL><<<blocks, kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_scatter(const FusedParams &p, cudaStream_t st)
{
    const size_t smem = (3 * static_cast<size_t>(p.T.npad) + static_cast<size_t>(p.G.lc_max) * 32 + kWarps * 32) * sizeof(double);
    const long long blocks = static_cast<long long>(p.n_mtiles) * p.n_ptiles * p.n_tables_launch;
    if (blocks <= 0 || blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const unsigned nb = static_cast<unsigned>(blocks);
    const bool all = (p.G.mask & 0x1C00u) == 0x1C00u, contig = p.G.P_list == nullptr;
    if (contig) return all ? launch_scatter_t<true, true>(p, smem, nb, st) : launch_scatter_t<true, false>(p, smem, nb, st);
    return all ? launch_scatter_t<false, true>(p, smem, nb, st) : launch_scatter_t<false, false>(p, smem, nb, st);
}

}  // namespace plogp
