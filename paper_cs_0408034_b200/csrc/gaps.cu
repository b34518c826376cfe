// gaps_kernel: g(x) of Section 2 at every distinct argument of the lane <-> P kernels (decide_kernel,
// segmin_kernel), once per table: g(1) for the rendezvous handshake, g(s) of every candidate segment size
// and g(m) of every message size.  The CTAs of those kernels that share a table (one per group of message
// sizes and tile of process counts) then read the values instead of staging the table and interpolating
// them again.  One CTA per table; worth its launch only on grids with many CTAs per launch (the host decides).
#include "device_common.cuh"

namespace plogp {

constexpr int kGapsThreads = 128;

__global__ void __launch_bounds__(kGapsThreads) gaps_kernel(const GapsParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *s_tab = reinterpret_cast<double *>(smem_raw);
    const int table = p.table0 + blockIdx.x;
    stage_table(s_tab, p.T, table);
    __syncthreads();
    double *row = p.gaps + static_cast<size_t>(blockIdx.x) * p.stride;
    const int n = 1 + p.G.n_s + p.G.n_m;
    for (int i = threadIdx.x; i < n; i += kGapsThreads) {
        double x = 1.0;
        if (i > p.G.n_s) x = static_cast<double>(p.G.m_list[i - 1 - p.G.n_s]);
        else if (i > 0) x = static_cast<double>(s_at(p.G, i - 1));
        row[i] = gap_at(s_tab, p.T.npad, x);
    }
}

cudaError_t launch_gaps(const GapsParams &p, cudaStream_t st)
{
    const size_t smem = 3 * static_cast<size_t>(p.T.npad) * sizeof(double);
    cudaError_t e = cudaSuccess;
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(gaps_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    if (p.n_tables_launch <= 0) return cudaErrorInvalidConfiguration;
    gaps_kernel<<<static_cast<unsigned>(p.n_tables_launch), kGapsThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace plogp
