// Sensitivity of the segmented strategies of Table 1 to the segment size (Section 3.1 searches the size that
// minimises the model; the measured Segmented Chain of the paper's Fig. 1(b) used a fixed 8 kB):
//   surface_kernel   the model of ids 2, 5, 9 for every candidate segment size, [table][3][P][m][s]
//   fixed_kernel     the model with one fixed segment size (the whole message where it does not fit) and its
//                    ratio to the minimum over the candidates that plogp_predict found
//   boundary_kernel  where the selected strategy changes between neighbouring P or neighbouring m
// The three are plain streaming kernels (one model evaluation or one comparison per output element).
#include "device_common.cuh"

#include <algorithm>

namespace plogp {

// One CTA: one table, one message size, kSurfP consecutive process counts; threads <-> candidate sizes, so
// g(s), k and the line coefficients are computed once per candidate and serve 3 x kSurfP outputs, and every
// store is a run of consecutive s.
constexpr int kSurfP = 8;

__global__ void __launch_bounds__(256) surface_kernel(const SensParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    const int midx = blockIdx.x % p.G.n_m, pchunk = blockIdx.x / p.G.n_m, trel = blockIdx.y;
    const int table = p.table0 + trel;
    stage_table(s_tab, p.T, table);
    __syncthreads();
    const double L = p.T.lat[table];
    const uint32_t m_u = p.G.m_list[midx];
    const uint32_t mask = p.G.mask;
    const int n_s = p.G.n_s, n_P = p.G.n_P, n_m = p.G.n_m;
    const int p0 = pchunk * kSurfP, p1 = min(p0 + kSurfP, n_P);
    const double nan = CUDART_NAN;
    for (int si = threadIdx.x; si < n_s; si += blockDim.x) {
        const uint32_t s = s_at(p.G, si);
        const bool fits = s <= m_u;
        double B = nan, C = nan, Q = nan;
        if (fits) {
            const double gs = gap_at(s_tab, p.T.npad, static_cast<double>(s));
            const double k = static_cast<double>(segments(m_u, s, p.G.k_mode));
            B = gs + L;
            C = gs * (k - 1.0);
            Q = gs * k;
        }
        for (int pi = p0; pi < p1; ++pi) {
            const int P = P_at(p.G, pi);
            const double pm1 = static_cast<double>(P - 1);
            const size_t o = ((static_cast<size_t>(table - p.out_table0) * 3 * n_P + pi) * n_m + midx) * n_s + si;
            const size_t plane = static_cast<size_t>(n_P) * n_m * n_s;
            if ((mask >> 2) & 1u) p.surface[o] = fits ? fma(pm1, Q, L) : nan;                      // (P-1) (g(s) k) + L
            if ((mask >> 5) & 1u) p.surface[o + plane] = fits ? fma(pm1, B, C) : nan;              // (P-1) (g(s)+L) + g(s)(k-1)
            if ((mask >> 9) & 1u)                                                                  // floor(log2 P) g(s) k + ceil(log2 P) L
                p.surface[o + 2 * plane] = fits ? fma(static_cast<double>(31 - __clz(P)), Q, static_cast<double>(32 - __clz(P - 1)) * L) : nan;
        }
    }
}

// One CTA: one table, 32 consecutive message sizes (lanes), a chunk of process counts (warps stride over it).
__global__ void __launch_bounds__(256) fixed_kernel(const SensParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    const int n_mtiles = (p.G.n_m + 31) / 32;
    const int mtile = blockIdx.x % n_mtiles, pchunk = blockIdx.x / n_mtiles, trel = blockIdx.y;
    const int table = p.table0 + trel;
    stage_table(s_tab, p.T, table);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int midx = mtile * 32 + lane;
    if (midx >= p.G.n_m) return;  // no barriers below
    const double L = p.T.lat[table];
    const uint32_t m_u = p.G.m_list[midx];
    // the fixed size where it fits, else the whole message in one segment (Section 3.1)
    const uint32_t s_eff = p.s_fixed <= m_u ? p.s_fixed : m_u;
    const double gs = gap_at(s_tab, p.T.npad, static_cast<double>(s_eff));
    const double k = static_cast<double>(segments(m_u, s_eff, p.G.k_mode));
    const double B = gs + L, C = gs * (k - 1.0), Q = gs * k;
    const uint32_t mask = p.G.mask;
    const int n_P = p.G.n_P, n_m = p.G.n_m;
    const size_t plane = static_cast<size_t>(n_P) * n_m;
    const int p0 = pchunk * p.p_per_cta, p1 = min(p0 + p.p_per_cta, n_P);
    for (int pi = p0 + warp; pi < p1; pi += n_warps) {
        const int P = P_at(p.G, pi);
        const double pm1 = static_cast<double>(P - 1);
        const size_t cell = static_cast<size_t>(pi) * n_m + midx;
        const size_t o3 = static_cast<size_t>(table - p.out_table0) * 3 * plane + cell;
        const size_t o13 = static_cast<size_t>(table - p.out_table0) * 13 * plane + cell;
        double t[3];
        t[0] = fma(pm1, Q, L);
        t[1] = fma(pm1, B, C);
        t[2] = fma(static_cast<double>(31 - __clz(P)), Q, static_cast<double>(32 - __clz(P - 1)) * L);
        const int ids[3] = {2, 5, 9};
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            if (!((mask >> ids[q]) & 1u)) continue;
            p.time_fixed[o3 + q * plane] = t[q];
            if (p.ratio) p.ratio[o3 + q * plane] = t[q] / p.pred_time[o13 + ids[q] * plane];
        }
    }
}

__global__ void boundary_kernel(const uint8_t *strategy, uint8_t *boundary, long long n_planes, int n_P, int n_m)
{
    const long long total = n_planes * n_P * n_m;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int im = static_cast<int>(i % n_m), ip = static_cast<int>((i / n_m) % n_P);
        const uint8_t s = strategy[i];
        uint8_t b = 0;
        if (ip + 1 < n_P && strategy[i + n_m] != s) b |= 1;  // the next larger process count selects another strategy
        if (im + 1 < n_m && strategy[i + 1] != s) b |= 2;    // the next larger message size does
        boundary[i] = b;
    }
}

// The same, eight consecutive message sizes per thread (n_m a multiple of 8, both arrays 8-byte aligned):
// one 8-byte load of the row, one of the next row, one 8-byte store.
__global__ void boundary8_kernel(const uint8_t *strategy, uint8_t *boundary, long long n_planes, int n_P, int n_m)
{
    const int groups = n_m >> 3;
    const long long total = n_planes * n_P * groups;
    for (long long gidx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; gidx < total;
         gidx += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int g = static_cast<int>(gidx % groups), ip = static_cast<int>((gidx / groups) % n_P);
        const long long i = (gidx / groups) * n_m + 8LL * g;
        const unsigned long long row = *reinterpret_cast<const unsigned long long *>(strategy + i);
        const unsigned long long below = ip + 1 < n_P ? *reinterpret_cast<const unsigned long long *>(strategy + i + n_m) : row;
        // the right neighbours: this group shifted by one byte, its last byte taken from the next group (or itself
        // at the end of the row, which has no neighbour)
        const unsigned long long last = g + 1 < groups ? strategy[i + 8] : (row >> 56);
        const unsigned long long right = (row >> 8) | (last << 56);
        unsigned long long out = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const unsigned long long sh = 8ull * b;
            const unsigned f = (((row >> sh) & 0xFF) != ((below >> sh) & 0xFF) ? 1u : 0u) |
                               (((row >> sh) & 0xFF) != ((right >> sh) & 0xFF) ? 2u : 0u);
            out |= static_cast<unsigned long long>(f) << sh;
        }
        *reinterpret_cast<unsigned long long *>(boundary + i) = out;
    }
}

cudaError_t launch_surface(const SensParams &p, cudaStream_t st)
{
    const size_t smem = 3 * static_cast<size_t>(p.T.npad) * sizeof(double);
    const long long bx = static_cast<long long>(p.G.n_m) * ((p.G.n_P + kSurfP - 1) / kSurfP);
    if (bx <= 0 || bx > 0x7FFFFFFFLL || p.n_tables_launch <= 0 || p.n_tables_launch > 65535) return cudaErrorInvalidConfiguration;
    const int threads = std::min(256, std::max(32, (p.G.n_s + 31) / 32 * 32));
    dim3 grid(static_cast<unsigned>(bx), static_cast<unsigned>(p.n_tables_launch));
    surface_kernel<<<grid, threads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_fixed(const SensParams &p, cudaStream_t st)
{
    const size_t smem = 3 * static_cast<size_t>(p.T.npad) * sizeof(double);
    const long long bx = static_cast<long long>((p.G.n_m + 31) / 32) * ((p.G.n_P + p.p_per_cta - 1) / p.p_per_cta);
    if (bx <= 0 || bx > 0x7FFFFFFFLL || p.n_tables_launch <= 0 || p.n_tables_launch > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(bx), static_cast<unsigned>(p.n_tables_launch));
    fixed_kernel<<<grid, 256, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_boundaries(const uint8_t *d_strategy, uint8_t *d_boundary, long long n_planes, int n_P, int n_m, int sm_count, cudaStream_t st)
{
    const long long total = n_planes * n_P * n_m;
    if (total <= 0) return cudaSuccess;
    const bool wide = n_m % 8 == 0 && reinterpret_cast<uintptr_t>(d_strategy) % 8 == 0 && reinterpret_cast<uintptr_t>(d_boundary) % 8 == 0;
    const long long want = ((wide ? total / 8 : total) + 255) / 256;
    const unsigned blocks = static_cast<unsigned>(std::min<long long>(want, static_cast<long long>(sm_count) * 32));
    if (wide) boundary8_kernel<<<blocks, 256, 0, st>>>(d_strategy, d_boundary, n_planes, n_P, n_m);
    else boundary_kernel<<<blocks, 256, 0, st>>>(d_strategy, d_boundary, n_planes, n_P, n_m);
    return cudaGetLastError();
}

}  // namespace plogp
