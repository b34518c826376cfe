// barrier_kernel: decision over the Barrier strategies.  The paper names the Barrier among the collectives that MPI
// implementations build like a Broadcast (Section 3) but prints no model for it; here a Barrier is a Reduce followed
// by a Broadcast of one-byte messages over the same tree, g(1) being the gap that Table 1's rendezvous rows use for an
// empty message:
//   23 Flat Tree      2 ((P-1) g(1) + L)
//   24 Chain          2 (P-1) (g(1) + L)
//   25 Binary Tree    2 ceil(log2 P) (2 g(1) + L)
//   26 Binomial Tree  2 (floor(log2 P) g(1) + ceil(log2 P) L)
// One decision per (table, P): microseconds of work, one thread per cell.  (Gather and Reduce, the other derived
// collectives, are the mirrored Scatter / Broadcast strategies and go through the decision kernels themselves.)
#include "device_common.cuh"

namespace plogp {

__global__ void barrier_kernel(TableDev T, GridDev G, int table0, int n_tables_launch, uint8_t *d_strategy, uint32_t *d_sbytes,
                               double *d_time)
{
    const long long total = static_cast<long long>(n_tables_launch) * G.n_P;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int trel = static_cast<int>(i / G.n_P), pidx = static_cast<int>(i % G.n_P);
        const int table = table0 + trel;
        const double *tab = T.tab + static_cast<size_t>(table) * 3 * T.npad;
        const double L = T.lat[table];
        // g(1): the table is read in place (global memory): below the first size its first value, else its line
        const double g1 = gap_at(tab, T.npad, 1.0);
        const int P = P_at(G, pidx);
        const double pm1 = static_cast<double>(P - 1), lf = static_cast<double>(31 - __clz(P)), lc = static_cast<double>(32 - __clz(P - 1));
        double bt = CUDART_INF;
        int bid = 255;
        auto consider = [&](int bit, int id, double t) {  // ascending id, strict '<': the lowest id stays on ties
            if (((G.mask >> bit) & 1u) && t < bt) { bt = t; bid = id; }
        };
        consider(0, 23, 2.0 * fma(pm1, g1, L));
        consider(3, 24, 2.0 * (pm1 * (g1 + L)));
        consider(6, 25, 2.0 * (lc * fma(2.0, g1, L)));
        consider(7, 26, 2.0 * fma(lf, g1, lc * L));
        const size_t o = static_cast<size_t>(table) * G.n_P + pidx;
        d_strategy[o] = static_cast<uint8_t>(bid);
        d_sbytes[o] = 0u;
        d_time[o] = bt;
    }
}

cudaError_t launch_barrier(const TableDev &T, const GridDev &G, int table0, int n_tables_launch, uint8_t *d_strategy, uint32_t *d_sbytes,
                           double *d_time, cudaStream_t st)
{
    const long long total = static_cast<long long>(n_tables_launch) * G.n_P;
    if (total <= 0) return cudaSuccess;
    const unsigned blocks = static_cast<unsigned>(total + 255 < 256LL * 4096 ? (total + 255) / 256 : 4096);
    barrier_kernel<<<blocks, 256, 0, st>>>(T, G, table0, n_tables_launch, d_strategy, d_sbytes, d_time);
    return cudaGetLastError();
}

}  // namespace plogp
