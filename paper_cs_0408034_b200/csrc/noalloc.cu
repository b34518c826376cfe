// plogp_scatter_chain_static: the Scatter Chain model (Table 2, second row) for callers that
// cannot allocate device memory.  It is a self-contained variant of the reduce-then-scan that the
// main path runs for this model; the per-tile partial sums, which the main path keeps in scratch
// it allocates, live here in one fixed array that is part of the library image.
//
// The array is shared by every call on a device and keeps whatever the last call left in it.
// Nothing in it has to start at zero: phase 1 writes every entry that phases 2 and 3 of the same
// call read.  Two calls whose device work overlaps would overwrite each other's partial sums.
#include "../../include/plogp.h"

#include <cuda_runtime.h>
#include <cmath>
#include <mutex>

namespace {

constexpr int kNaThreads = 256;
constexpr int kNaWarps = kNaThreads / 32;
constexpr int kNaR = 4;                              // process counts per thread and pass
constexpr int kNaPassP = kNaWarps * kNaR;            // 32 process counts per pass
constexpr int kNaPasses = 32;                        // passes per tile
constexpr int kNaTileP = kNaPassP * kNaPasses;       // 1024 process counts per tile
constexpr int kNaMaxM = PLOGP_STATIC_MAX_M;          // message sizes
constexpr int kNaMaxTiles = PLOGP_STATIC_MAX_P / kNaTileP;
constexpr int kNaScratchDoubles = kNaMaxTiles * kNaMaxM;  // 65536 doubles = 512 KiB
constexpr int kMaxDevices = 64;

// Partial sums [tile][m].  In host code this name is only a handle for the runtime; the device
// address is fetched once per device with cudaGetSymbolAddress and passed to the kernels.
static __device__ __align__(256) double g_static_scratch[kNaScratchDoubles];

// The scan runs over the terms j = 1 .. P_hi - 1 of the sum, whatever P_lo is: term index e stands for j = e + 1,
// i.e. for the process count P = e + 2, and rows below P_lo are simply not written.  All CTAs share the work
// for the terms below P_lo that way, and no thread ever owns more than one term per index.
struct NaArgs {
    const uint64_t *sizes;
    const double *gap;
    const uint64_t *m;
    double *time;
    double *scratch;
    double L;
    int n_bp, npad, P_lo, n_terms, n_m, n_mtiles, n_ptiles;
};

// key | gap | slope in shared memory, built from the caller's raw table
__device__ void na_stage(double *s_tab, const NaArgs &a)
{
    for (int i = threadIdx.x; i < a.npad; i += blockDim.x) {
        double key = __longlong_as_double(0x7FF0000000000000LL), g = 0.0, sl = 0.0;
        if (i <= a.n_bp - 2) {
            key = static_cast<double>(a.sizes[i]);
            g = a.gap[i];
            sl = (a.gap[i + 1] - g) / static_cast<double>(a.sizes[i + 1] - a.sizes[i]);
        }
        s_tab[i] = key;
        s_tab[a.npad + i] = g;
        s_tab[2 * a.npad + i] = sl;
    }
}

// g(x) of Section 2 (piecewise linear, held below the table, last line continued above it)
__device__ __forceinline__ double na_gap(const double *s_tab, int npad, double x)
{
    int i = 0;
    for (int step = npad >> 1; step > 0; step >>= 1) {
        const int j = i + step;
        i = (s_tab[j] <= x) ? j : i;
    }
    return fma(fmax(x - s_tab[i], 0.0), s_tab[2 * npad + i], s_tab[npad + i]);
}

// PHASE 1: per-tile sums of g(j m) into the scratch.  PHASE 3: prefix over P with the scanned
// tile sums as carry, written out as sum + (P-1) L.
template <int PHASE>
__global__ void __launch_bounds__(kNaThreads) na_chain_kernel(const NaArgs a)
{
    extern __shared__ __align__(16) unsigned char na_smem[];
    double *s_tab = reinterpret_cast<double *>(na_smem);
    double *s_tot = s_tab + 3 * a.npad;  // [2][warps][32]

    const int mtile = blockIdx.x % a.n_mtiles, ptile = blockIdx.x / a.n_mtiles;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int midx = mtile * 32 + lane;
    const bool m_ok = midx < a.n_m;
    const double md = static_cast<double>(a.m[min(midx, a.n_m - 1)]);

    na_stage(s_tab, a);
    __syncthreads();

    double carry = (PHASE == 3 && m_ok) ? a.scratch[ptile * a.n_m + midx] : 0.0;
    double acc = 0.0;
    for (int pass = 0; pass < kNaPasses; ++pass) {
        const int e_cta = ptile * kNaTileP + pass * kNaPassP;
        if (e_cta >= a.n_terms) break;
        const int e0 = e_cta + warp * kNaR;
        double pre[kNaR];
        double run = 0.0;
#pragma unroll
        for (int r = 0; r < kNaR; ++r) {
            const int e = e0 + r;
            if (e < a.n_terms) run += na_gap(s_tab, a.npad, static_cast<double>(e + 1) * md);  // g(j m), j = e + 1
            pre[r] = run;
        }
        if (PHASE == 1) {
            acc += run;
        } else {
            double *tot = s_tot + (pass & 1) * (kNaWarps * 32);
            tot[warp * 32 + lane] = run;
            __syncthreads();
            double before = 0.0, all = 0.0;
#pragma unroll
            for (int w = 0; w < kNaWarps; ++w) {
                const double v = tot[w * 32 + lane];
                before += (w < warp) ? v : 0.0;
                all += v;
            }
#pragma unroll
            for (int r = 0; r < kNaR; ++r) {
                const int e = e0 + r;
                const int P = e + 2;  // the sum up to j = e + 1 = P - 1 belongs to this process count
                if (e < a.n_terms && P >= a.P_lo && m_ok)
                    a.time[static_cast<size_t>(P - a.P_lo) * a.n_m + midx] =
                        fma(static_cast<double>(P - 1), a.L, carry + before + pre[r]);
            }
            carry += all;
        }
    }
    if (PHASE == 1) {
        s_tot[warp * 32 + lane] = acc;
        __syncthreads();
        if (warp == 0 && m_ok) {
            double t = 0.0;
#pragma unroll
            for (int w = 0; w < kNaWarps; ++w) t += s_tot[w * 32 + lane];
            a.scratch[ptile * a.n_m + midx] = t;
        }
    }
}

// PHASE 2: exclusive scan of the tile sums along the tile index, in place
__global__ void na_scan_kernel(double *scratch, int n_ptiles, int n_m)
{
    const int midx = blockIdx.x * blockDim.x + threadIdx.x;
    if (midx >= n_m) return;
    double run = 0.0;
    for (int pt = 0; pt < n_ptiles; ++pt) {
        const double v = scratch[pt * n_m + midx];
        scratch[pt * n_m + midx] = run;
        run += v;
    }
}

std::mutex g_setup_mutex;
double *g_scratch_addr[kMaxDevices] = {};

}  // namespace

extern "C" int plogp_scatter_chain_static(int n_bp, const uint64_t *d_sizes_bytes, const double *d_gap,
                                          double latency, int32_t P_lo, int32_t P_hi,
                                          const uint64_t *d_m_bytes, int32_t n_m, double *d_time, void *stream)
{
    if (!d_sizes_bytes || !d_gap || !d_m_bytes || !d_time) return PLOGP_E_INVAL;
    if (n_bp < 2 || P_lo < 2 || P_hi < P_lo || n_m < 1 || !std::isfinite(latency) || latency < 0.0) return PLOGP_E_INVAL;
    const long long n_terms = static_cast<long long>(P_hi) - 1;  // j = 1 .. P_hi - 1
    if (n_bp > PLOGP_MAX_BREAKPOINTS || n_m > PLOGP_STATIC_MAX_M || n_terms > PLOGP_STATIC_MAX_P) return PLOGP_E_RANGE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PLOGP_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return PLOGP_E_RANGE;
    double *scratch = nullptr;
    {
        // One-time set-up per device, with that device current: turn the symbol into an address.
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
                cudaGetLastError();
                return PLOGP_E_CUDA;
            }
            g_scratch_addr[dev] = static_cast<double *>(p);
        }
        scratch = g_scratch_addr[dev];
    }

    NaArgs a{};
    a.sizes = d_sizes_bytes; a.gap = d_gap; a.m = d_m_bytes; a.time = d_time; a.scratch = scratch;
    a.L = latency; a.n_bp = n_bp; a.P_lo = P_lo; a.n_terms = static_cast<int>(n_terms); a.n_m = n_m;
    a.npad = 2;
    while (a.npad < n_bp - 1) a.npad <<= 1;
    a.n_mtiles = (n_m + 31) / 32;
    a.n_ptiles = (a.n_terms + kNaTileP - 1) / kNaTileP;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = (3 * static_cast<size_t>(a.npad) + 2 * kNaWarps * 32) * sizeof(double);  // <= 28 KiB
    const unsigned blocks = static_cast<unsigned>(a.n_mtiles * a.n_ptiles);
    na_chain_kernel<1><<<blocks, kNaThreads, smem, st>>>(a);
    na_scan_kernel<<<(n_m + 127) / 128, 128, 0, st>>>(scratch, a.n_ptiles, n_m);
    na_chain_kernel<3><<<blocks, kNaThreads, smem, st>>>(a);
    return cudaGetLastError() == cudaSuccess ? PLOGP_OK : PLOGP_E_CUDA;
}
