// Internal declarations shared by the host side (api.cu) and the kernels (kernels.cu).
// Nothing here is part of the public ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace plogp {

// Tables as they live in device memory.  Per table: three runs of `npad` doubles
//   key[npad]   breakpoint sizes usable as interval starts (index <= n_bp-2), +inf beyond
//   gap[npad]   g at the interval start
//   slope[npad] (g[i+1]-g[i]) / (size[i+1]-size[i])
// npad is a power of two >= n_bp, so the interval search needs no bounds checks and an upward
// walk always meets a +inf key.
// Where a decision kernel puts its results and how it names the strategies.  plogp_select_best writes two planes
// per table (Broadcast, Scatter) with the ids of Table 1 / Table 2; the derived collectives (Gather, Reduce) reuse
// the same kernels with one plane per table and the ids of the mirrored strategies.
struct OutMap {
    int planes;       // decision planes per table in the output arrays
    int plane_bcast;  // plane that receives the Broadcast-type decision
    int plane_scat;   // plane that receives the Scatter-type decision
    uint8_t id_of[16];  // output id of internal strategy id 0..12 (255 beyond)
};

struct TableDev {
    const double *tab;  // [n_tables][3*npad]
    const double *lat;  // [n_tables]
    int n_tables, n_bp, npad;
};

struct GridDev {
    const int32_t *P_list;  // device [n_P] or nullptr => P = P_lo + index
    int n_P, P_lo;
    const uint32_t *m_list;  // device [n_m]
    int n_m;
    const uint32_t *s_list;  // device [n_s] or nullptr => s = s_lo + index * s_step
    int n_s;
    uint32_t s_lo, s_step;
    const int32_t *ns_of_m;  // device [n_m]: number of candidates s <= m (0 => unsegmented fallback)
    const double *k_list;    // device [n_m][n_s]: Section 2's k for every (m, candidate s <= m), short candidate lists only
    uint32_t mask;
    int k_mode;
    int lc_max;  // ceil(log2 P_hi)
};

// Segment-sweep kernel (large candidate lists): partial minima per (table, segmented strategy,
// (m, chunk) pair, P).
struct SweepParams {
    TableDev T;
    GridDev G;
    const int32_t *pair_m;      // device [n_pairs] in launch order (heaviest first)
    const int32_t *pair_chunk;  // device [n_pairs]
    const int32_t *pair_row;    // device [n_pairs]: row id of the pair (= pair_base[m] + chunk)
    int n_pairs, n_ptiles, chunk_len;
    double *part_time;   // [n_tables_batch][n_seg][n_pairs][n_P]
    uint32_t *part_idx;  // same shape: index of s in the candidate list
    int n_seg;           // enabled segmented strategies (slots in id order)
    int table0;          // first table of this launch (blockIdx.y is relative to it)
};

// Envelope kernel (exact fast path of the segment-size search): same scratch layout as the sweep kernel with
// one row per message size.
struct EnvParams {
    TableDev T;
    GridDev G;
    int table0, n_tables_launch;
    double *part_time;   // [n_tables_batch][n_seg][n_m][n_P]
    uint32_t *part_idx;  // same shape: index of s in the candidate list
    int n_seg;
    int rep_cap;     // entries of the shared-memory list of representatives (longer lists go through it in windows)
    int coarse;      // distance between the coarse process-count indices
    int max_coarse;  // capacity of the coarse-winner array (>= number of coarse indices)
};

// Segment-size sensitivity kernels (sensitivity.cu)
struct SensParams {
    TableDev T;
    GridDev G;
    int table0, n_tables_launch, out_table0;
    double *surface;           // [n_tables][3][n_P][n_m][n_s]
    uint32_t s_fixed;          // the fixed segment size (fixed_kernel)
    int p_per_cta;             // process counts per CTA (fixed_kernel)
    const double *pred_time;   // [n_tables][13][n_P][n_m] from plogp_predict, or nullptr together with ratio
    double *time_fixed, *ratio;  // [n_tables][3][n_P][n_m]
};

struct FusedParams {
    TableDev T;
    GridDev G;
    int n_mtiles, n_ptiles, passes_per_tile;  // a pass covers kWarps*R process counts
    int table0, n_tables_launch;
    int out_table0;  // table whose results sit at the start of the output arrays (0 unless the caller passes a window)
    OutMap om;
    const double *s1_sums;  // [n_tables_launch][n_ptiles][9][n_m] Scatter Chain sums per warp run and per tile, or nullptr
    // segmented minima precomputed by the sweep kernel (nullptr => inline sweep)
    const double *part_time;
    const uint32_t *part_idx;
    const int32_t *pair_base;  // device [n_m+1]
    int n_pairs, n_seg;
    // outputs: decision table
    uint8_t *d_strategy;
    uint32_t *d_sbytes;
    double *d_time;
    // outputs: predicted planes
    double *p_time;
    uint32_t *p_best_s;
};

struct S1Params {
    TableDev T;
    GridDev G;
    int n_mtiles, n_ptiles, passes_per_tile;
    int table0, n_tables_launch;
    double *tile_sum;  // [n_tables_launch][n_ptiles][9][n_m]: the 8 warps' shares, then the tile's total
};

// Gap pre-pass (gaps.cu): g at every distinct argument of the lane <-> P kernels, once per table.
// Row of a table: [0] = g(1), [1 .. n_s] = g(s_i), [1 + n_s .. 1 + n_s + n_m) = g(m_j).
struct GapsParams {
    TableDev T;
    GridDev G;
    int table0, n_tables_launch;
    double *gaps;  // [n_tables_launch][stride]
    int stride;
};

// Decision kernel for short candidate lists (lanes <-> P): see decide.cu
struct DecideParams {
    TableDev T;
    GridDev G;
    const double *gaps;  // rows of the gap pre-pass for this launch's tables, or nullptr: the kernel interpolates itself
    int gaps_stride;
    int n_mgroups, n_ptiles;
    int mg;  // message sizes per CTA, 1..kDecMG
    int envelope;  // lower-envelope search: the lists keep only the candidates that can win (see decide.cu)
    int vec_out;  // outputs aligned for two message sizes per store (n_m even, 16 / 8 / 2-byte aligned bases)
    int table0, n_tables_launch;
    int out_table0;  // table whose results sit at the start of the output arrays
    OutMap om;
    uint8_t *d_strategy;
    uint32_t *d_sbytes;
    double *d_time;
};

constexpr int kDecThreads = 128;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecR = 8;                               // process counts per thread
constexpr int kDecTileP = 32 * kDecR;                  // 256 process counts per CTA, shared by its warps
constexpr int kDecMG = 16;                             // message sizes per CTA (at most), split over the warps
constexpr int kDecU = 4;                               // list entries per filter test

// segmin_kernel (segmented minima of plogp_predict on short candidate lists, lanes <-> P): see segmin.cu
struct SegminParams {
    TableDev T;
    GridDev G;
    const double *gaps;  // as in DecideParams
    int gaps_stride;
    int vec_out;  // outputs aligned for two message sizes per store (n_m even, 16-byte aligned times, 8-byte aligned sizes)
    int n_mgroups, n_ptiles;
    int table0, n_tables_launch, out_table0;
    double *p_time;      // [n_tables][13][n_P][n_m]: planes 2, 5, 9 are written
    uint32_t *p_best_s;  // [n_tables][3][n_P][n_m], or nullptr
};
constexpr int kSegThreads = 256;
constexpr int kSegWarps = kSegThreads / 32;
constexpr int kSegR = 8;                 // process counts per thread
constexpr int kSegTileP = 32 * kSegR;    // process counts per CTA
constexpr int kSegMG = 16;               // message sizes per CTA, two per warp

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kFusedR = 4;   // process counts per thread and pass in the fused kernel
constexpr int kSweepR = 8;   // process counts per thread in the sweep kernel
constexpr int kSweepSub = 256;  // candidates staged per sub-chunk
constexpr int kSweepU = 4;      // candidates per filter test in the sweep kernel
constexpr int kMaxInlineS = 64;

size_t fused_smem_bytes(const TableDev &T, const GridDev &G, bool inline_sweep);
cudaError_t launch_fused(const FusedParams &p, bool predict, cudaStream_t st);
cudaError_t launch_scatter(const FusedParams &p, cudaStream_t st);  // decision table, Scatter strategies only
cudaError_t launch_sweep(const SweepParams &p, int n_tables_launch, cudaStream_t st);
cudaError_t launch_s1_tiles(const S1Params &p, cudaStream_t st);
size_t decide_smem_bytes(const TableDev &T, const GridDev &G);
cudaError_t launch_decide(const DecideParams &p, cudaStream_t st);
cudaError_t launch_fp64_probe(double *d_sink, int iters, int blocks, cudaStream_t st);
size_t segmin_smem_bytes(const TableDev &T, const GridDev &G);
cudaError_t launch_segmin(const SegminParams &p, cudaStream_t st);
cudaError_t launch_gaps(const GapsParams &p, cudaStream_t st);
cudaError_t launch_barrier(const TableDev &T, const GridDev &G, int table0, int n_tables_launch, uint8_t *d_strategy, uint32_t *d_sbytes,
                           double *d_time, cudaStream_t st);
cudaError_t launch_surface(const SensParams &p, cudaStream_t st);
cudaError_t launch_fixed(const SensParams &p, cudaStream_t st);
cudaError_t launch_boundaries(const uint8_t *d_strategy, uint8_t *d_boundary, long long n_planes, int n_P, int n_m, int sm_count, cudaStream_t st);
size_t envelope_smem_bytes(const TableDev &T, int threads, int rep_cap, int max_coarse);
cudaError_t launch_envelope(const EnvParams &p, int threads, cudaStream_t st);

}  // namespace plogp
