// Device helpers shared by the kernels: table staging into shared memory, g(x), grid accessors.
#pragma once

#include "internal.h"

#include <math_constants.h>

namespace plogp {

// ------------------------------------------------------------------------------------------
// Table staging and g(x)
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src));
}

__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n" ::: "memory");
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}

// Copies one table (key | gap | slope, 3*npad doubles) into shared memory with 16-byte
// asynchronous copies.  The caller synchronises the CTA afterwards.
__device__ __forceinline__ void stage_table(double *s_tab, const TableDev &T, int table)
{
    const double *src = T.tab + static_cast<size_t>(table) * 3 * T.npad;
    const int n16 = (3 * T.npad) >> 1;
    for (int i = threadIdx.x; i < n16; i += blockDim.x) cp_async16(s_tab + 2 * i, src + 2 * i);
    cp_async_wait_all();
}

// g(x) of Section 2 on the staged table: branch-free search of the interval that starts at or
// below x (keys beyond the last interval are +inf), then one fused multiply-add along that
// interval's line.  x below the first size is held at the first gap (dx clamped to 0); x above
// the last size continues the last interval's line.
__device__ __forceinline__ double gap_at(const double *s_tab, int npad, double x)
{
    int i = 0;
#pragma unroll 1
    for (int step = npad >> 1; step > 0; step >>= 1) {
        const int j = i + step;
        i = (s_tab[j] <= x) ? j : i;
    }
    const double dx = fmax(x - s_tab[i], 0.0);
    return fma(dx, s_tab[2 * npad + i], s_tab[npad + i]);
}

__device__ __forceinline__ int P_at(const GridDev &G, int pidx)
{
    return G.P_list ? G.P_list[pidx] : G.P_lo + pidx;
}

__device__ __forceinline__ uint32_t s_at(const GridDev &G, int si)
{
    return G.s_list ? G.s_list[si] : G.s_lo + static_cast<uint32_t>(si) * G.s_step;
}

// k of Section 2: number of segments of size s in a message of m bytes.
__device__ __forceinline__ uint32_t segments(uint32_t m, uint32_t s, int k_mode)
{
    const uint32_t q = m / s;
    return q + ((k_mode == 0 && q * s != m) ? 1u : 0u);
}

// Interval search alone: largest i with key[i] <= x (0 when x is below the table).
__device__ __forceinline__ int interval_of(const double *s_tab, int npad, double x)
{
    int i = 0;
#pragma unroll 1
    for (int step = npad >> 1; step > 0; step >>= 1) {
        const int j = i + step;
        i = (s_tab[j] <= x) ? j : i;
    }
    return i;
}

// g(x) for a caller whose arguments never decrease: the current interval's line is kept in
// registers and shared memory is touched only when x crosses into the next interval (keys past
// the last interval are +inf, and npad >= n_bp leaves at least one such key, so the walk stops
// inside the array).
struct GapWalk {
    int i = -1;
    double key, next, slope, gap;

    __device__ __forceinline__ void load(const double *s_tab, int npad)
    {
        key = s_tab[i];
        next = s_tab[i + 1];
        slope = s_tab[2 * npad + i];
        gap = s_tab[npad + i];
    }
    __device__ __forceinline__ double at(const double *s_tab, int npad, double x)
    {
        if (i < 0) {
            i = interval_of(s_tab, npad, x);
            load(s_tab, npad);
        }
        while (x >= next) {
            ++i;
            load(s_tab, npad);
        }
        return fma(fmax(x - key, 0.0), slope, gap);
    }
};

// Lexicographic minimum of (t, e) over a warp (all lanes receive it).
__device__ __forceinline__ void warp_min_pair(double &t, int &e)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double t2 = __shfl_xor_sync(0xffffffffu, t, off);
        const int e2 = __shfl_xor_sync(0xffffffffu, e, off);
        if (t2 < t || (t2 == t && e2 < e)) { t = t2; e = e2; }
    }
}

// Sum of g(j m) for j = jlo .. jhi (jlo <= jhi) in closed form: inside one table interval g is a line, so the
// terms whose arguments fall into it are an arithmetic series, n gap_i + slope_i (m (jlo' + jhi') n / 2 - n key_i);
// the loop runs over the table intervals that the arguments cross (at most n_bp), not over j.  Below the first
// size g is constant (its first value), above the last size the last interval's line goes on.  This is what
// keeps a gap in a process-count list, or a first process count far above 2, from turning into a long loop.
static __device__ __noinline__ double chain_range_sum(const double *s_tab, int npad, double md, long long jlo, long long jhi)
{
    double sum = 0.0;
    long long j = jlo;
    int i = -1;  // -1: below the table
    if (static_cast<double>(j) * md >= s_tab[0]) i = interval_of(s_tab, npad, static_cast<double>(j) * md);
    while (j <= jhi) {
        const double next = s_tab[i + 1];  // first argument that belongs to the next interval (+inf after the last)
        long long jend = jhi;
        if (next <= static_cast<double>(jhi) * md) {
            // largest j with j m < next (m, next and the products are integers below 2^53: exact)
            long long q = static_cast<long long>(next / md);
            while (static_cast<double>(q) * md >= next) --q;
            while (static_cast<double>(q + 1) * md < next) ++q;
            jend = q;
        }
        if (jend >= j) {
            const double n = static_cast<double>(jend - j + 1);
            if (i < 0) {
                sum += n * s_tab[npad];
            } else {
                const double mean = 0.5 * (static_cast<double>(j + jend) * md) - s_tab[i];  // mean argument minus the key
                sum += n * fma(mean, s_tab[2 * npad + i], s_tab[npad + i]);
            }
            j = jend + 1;
        }
        ++i;
    }
    return sum;
}

// One term of the Scatter Chain sum for the process count at index pidx: the gaps g(j m) for j
// from the previous listed process count (1 before the first) up to P-1.  For a contiguous
// range of P this is the single gap g((P-1) m); longer runs are summed interval by interval.
// The walk state must only see non-decreasing arguments.
__device__ __forceinline__ double s1_term(const double *s_tab, int npad, const GridDev &G, int pidx, double md, GapWalk &w)
{
    const int jhi = P_at(G, pidx) - 1;
    const int jlo = pidx == 0 ? 1 : P_at(G, pidx - 1);
    if (jlo == jhi) return w.at(s_tab, npad, static_cast<double>(jlo) * md);
    return chain_range_sum(s_tab, npad, md, jlo, jhi);
}

// Scatter Chain sum in front of a warp's run when the P range is split over CTAs: the totals of the tiles
// in front of this one (added up by the CTA's warps in a fixed order: warp w takes tiles w, w + 8, ...) plus
// the shares of the lower warps of this tile.  sums is laid out [table][tile][9][m] (8 warp shares, then the
// tile's total); s_buf holds kWarps * 32 doubles.  Called by all threads of the CTA (one barrier inside).
__device__ __forceinline__ double chain_prefix(const double *sums, int trel, int n_ptiles, int ptile, int warp, int lane,
                                               int n_m, int midx_c, double *s_buf)
{
    const double *tab0 = sums + static_cast<size_t>(trel) * n_ptiles * (kWarps + 1) * n_m + midx_c;
    double part = 0.0;
    for (int t = warp; t < ptile; t += kWarps) part += tab0[(static_cast<size_t>(t) * (kWarps + 1) + kWarps) * n_m];
    s_buf[warp * 32 + lane] = part;
    __syncthreads();
    double run = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) run += s_buf[w * 32 + lane];
    const double *mine = tab0 + static_cast<size_t>(ptile) * (kWarps + 1) * n_m;
    for (int w = 0; w < warp; ++w) run += mine[static_cast<size_t>(w) * n_m];
    return run;
}

}  // namespace plogp
