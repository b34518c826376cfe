// Host side of the C ABI declared in include/plogp.h: argument validation, table upload, the
// launch plan for a grid (tiling, chunking of long candidate lists, scratch layout) and the
// kernel launches.  Every step of the evaluation itself runs in kernels.cu.
#include "../../include/plogp.h"
#include "internal.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <string>
#include <vector>

using namespace plogp;

namespace {

thread_local std::string g_cuda_error;
std::atomic<unsigned long long> g_launches{0};

int cuda_fail(cudaError_t e, const char *what)
{
    g_cuda_error = std::string(what) + ": " + cudaGetErrorName(e) + " (" + cudaGetErrorString(e) + ")";
    cudaGetLastError();  // clear the sticky-free error state
    return PLOGP_E_CUDA;
}

#define CK(call)                                                  \
    do {                                                          \
        cudaError_t e_ = (call);                                  \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);       \
    } while (0)

constexpr uint32_t kSegBits = (1u << 2) | (1u << 5) | (1u << 9);
constexpr uint64_t kTwo32 = 1ull << 32;
constexpr double kTwo53 = 9007199254740992.0;
constexpr int64_t kMaxP = int64_t(1) << 30;  // process counts: 32-bit tiling arithmetic and 1 << ceil(log2 P) stay in range
constexpr size_t kSweepScratchLimit = size_t(1) << 30;  // per launch batch of tables

int ceil_log2(int64_t P)
{
    int e = 0;
    while ((int64_t(1) << e) < P) ++e;
    return e;
}

// Everything derived from a grid that the launches need; cached on the handle while the same
// grid keeps being passed.
struct Plan {
    std::vector<unsigned char> key;  // serialised grid, for the cache comparison
    bool empty = true;
    GridDev G{};
    int n_seg = 0;
    bool inline_sweep = true;
    bool envelope = false;        // envelope_kernel instead of the sweep kernel (long candidate lists)
    bool envelope_short = false;  // the decision kernel prunes its candidate lists (short candidate lists)
    int env_threads = 256, env_rep_cap = 0, env_coarse = 64, env_max_coarse = 0;
    // fused kernel tiling
    int n_mtiles = 0, n_ptiles = 1, passes_per_tile = 1;
    // Scatter decision kernel: its own split of P (one CTA run covers a short P range in a few microseconds,
    // and an unsplit range needs no tile sums, i.e. one launch less)
    int sc_ptiles = 1, sc_passes_per_tile = 1;
    // decision kernel tiling (short candidate lists)
    int dec_mgroups = 0, dec_ptiles = 1, dec_mg = kDecMG;
    size_t carry_bytes_per_table = 0;
    // sweep kernel
    int n_pairs = 0, sweep_ptiles = 0, chunk_len = 0;
    size_t off_pair_m = 0, off_pair_chunk = 0, off_pair_row = 0, off_pair_base = 0;
    int tables_per_batch = 0;
    size_t scratch_bytes = 0;
    size_t off_k = 0;          // k table of the lane <-> P kernels inside the grid blob
    bool use_gaps = false;     // run the gap pre-pass in front of the lane <-> P kernels
    int gaps_stride = 0;       // doubles per table in its output
    size_t gaps_bytes_per_table = 0;
};

}  // namespace

struct plogp_tables {
    int device = 0;
    int sm_count = 148;
    TableDev T{};
    bool monotone = false;  // no table's gap ever decreases with the size (the envelope search relies on it)
    double *d_tab = nullptr, *d_lat = nullptr;
    unsigned char *d_grid = nullptr;
    size_t grid_cap = 0;
    unsigned char *d_ws = nullptr;
    size_t ws_cap = 0;
    Plan plan;
    // optional per-kernel timing: event pairs recorded around every launch while enabled
    // host-output path: two device staging sets and a copy stream
    unsigned char *d_stage[2] = {nullptr, nullptr};
    size_t stage_cap = 0;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_done[2] = {nullptr, nullptr}, ev_copied[2] = {nullptr, nullptr};
    bool profiling = false;
    struct Timed { int kind; cudaEvent_t a, b; };
    std::vector<Timed> timed;
};

namespace {

// Brackets one kernel launch with events on the caller's stream when timing is enabled.
struct LaunchTimer {
    plogp_tables *h;
    cudaStream_t st;
    cudaEvent_t a = nullptr, b = nullptr;
    int kind;
    LaunchTimer(plogp_tables *h_, int kind_, cudaStream_t st_) : h(h_), st(st_), kind(kind_)
    {
        if (!h->profiling) return;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess || cudaEventRecord(a, st) != cudaSuccess) {
            if (a) cudaEventDestroy(a);
            if (b) cudaEventDestroy(b);
            a = b = nullptr;
            cudaGetLastError();
        }
    }
    ~LaunchTimer()
    {
        if (!a) return;
        if (cudaEventRecord(b, st) == cudaSuccess) h->timed.push_back({kind, a, b});
        else { cudaEventDestroy(a); cudaEventDestroy(b); cudaGetLastError(); }
    }
};


template <typename V>
void put(std::vector<unsigned char> &buf, const V &v)
{
    const unsigned char *p = reinterpret_cast<const unsigned char *>(&v);
    buf.insert(buf.end(), p, p + sizeof(V));
}

template <typename V>
void put_array(std::vector<unsigned char> &buf, const V *v, size_t n)
{
    const unsigned char *p = reinterpret_cast<const unsigned char *>(v);
    buf.insert(buf.end(), p, p + n * sizeof(V));
}

template <typename V>
size_t append_aligned(std::vector<unsigned char> &blob, const std::vector<V> &v)
{
    while (blob.size() % 16) blob.push_back(0);
    const size_t off = blob.size();
    put_array(blob, v.data(), v.size());
    return off;
}

int validate_grid(const plogp_tables *h, const plogp_grid *g, int64_t *n_s_out)
{
    if (!g) return PLOGP_E_INVAL;
    if (g->strategy_mask >> PLOGP_N_STRATEGIES) return PLOGP_E_INVAL;
    if (g->k_mode != 0 && g->k_mode != 1) return PLOGP_E_INVAL;
    if (g->search_mode != 0 && g->search_mode != 1) return PLOGP_E_INVAL;
    if (g->dtype_bytes == 0) return PLOGP_E_INVAL;
    if (g->n_m < 0) return PLOGP_E_INVAL;
    if (g->n_m > 0 && !g->m) return PLOGP_E_INVAL;
    int64_t P_hi;
    if (g->P) {
        if (g->n_P < 0) return PLOGP_E_INVAL;
        for (int i = 0; i < g->n_P; ++i) {
            if (g->P[i] < 2) return PLOGP_E_INVAL;
            if (i && g->P[i] <= g->P[i - 1]) return PLOGP_E_INVAL;
        }
        P_hi = g->n_P ? g->P[g->n_P - 1] : 2;
    } else {
        if (g->P_lo < 2 || g->P_hi < g->P_lo) return PLOGP_E_INVAL;
        P_hi = g->P_hi;
    }
    if (P_hi > kMaxP) return PLOGP_E_RANGE;
    for (int i = 0; i < g->n_m; ++i) {
        const uint64_t m = g->m[i];
        if (m == 0 || m % g->dtype_bytes) return PLOGP_E_INVAL;
        if (i && m <= g->m[i - 1]) return PLOGP_E_INVAL;
        if (m >= kTwo32) return PLOGP_E_RANGE;
    }
    if (g->n_m > 0 && double(P_hi) * double(g->m[g->n_m - 1]) >= kTwo53) return PLOGP_E_RANGE;
    int64_t n_s = 0;
    if (g->strategy_mask & kSegBits) {
        if (g->s) {
            if (g->n_s < 0) return PLOGP_E_INVAL;
            for (int64_t i = 0; i < g->n_s; ++i) {
                const uint64_t s = g->s[i];
                if (s == 0 || s % g->dtype_bytes) return PLOGP_E_INVAL;
                if (i && s <= g->s[i - 1]) return PLOGP_E_INVAL;
                if (s >= kTwo32) return PLOGP_E_RANGE;
            }
            n_s = g->n_s;
        } else {
            if (g->s_step == 0 || g->s_step % g->dtype_bytes) return PLOGP_E_INVAL;
            if (g->s_lo == 0 || g->s_lo % g->dtype_bytes) return PLOGP_E_INVAL;
            if (g->s_hi >= g->s_lo) {
                if (g->s_hi >= kTwo32) return PLOGP_E_RANGE;
                n_s = int64_t((g->s_hi - g->s_lo) / g->s_step) + 1;
            }
        }
        if (n_s >= (int64_t(1) << 31)) return PLOGP_E_RANGE;
    }
    (void)h;
    *n_s_out = n_s;
    return PLOGP_OK;
}

// Builds (or reuses) the launch plan of a grid and makes its device arrays current.
int prepare(plogp_tables *h, const plogp_grid *g, cudaStream_t st)
{
    if (!g || g->n_m < 0 || (g->n_m > 0 && !g->m)) return PLOGP_E_INVAL;
    if (g->P && g->n_P < 0) return PLOGP_E_INVAL;
    if ((g->strategy_mask & kSegBits) && g->s && g->n_s < 0) return PLOGP_E_INVAL;
    // ---- cache key: every input that the plan depends on ----
    std::vector<unsigned char> key;
    key.reserve(256 + size_t(std::max(g->n_m, 0)) * 8);
    const int has_P = g->P != nullptr, has_s = g->s != nullptr;
    put(key, has_P);
    if (has_P) { put(key, g->n_P); put_array(key, g->P, size_t(std::max(g->n_P, 0))); }
    else { put(key, g->P_lo); put(key, g->P_hi); }
    put(key, g->n_m);
    put_array(key, g->m, size_t(std::max(g->n_m, 0)));
    put(key, g->strategy_mask); put(key, g->k_mode); put(key, g->dtype_bytes);
    put(key, g->search_mode); put(key, int(h->monotone));
    if (g->strategy_mask & kSegBits) {
        put(key, has_s);
        if (has_s) { put(key, g->n_s); put_array(key, g->s, size_t(std::max<int64_t>(g->n_s, 0))); }
        else { put(key, g->s_lo); put(key, g->s_hi); put(key, g->s_step); }
    }
    if (!h->plan.key.empty() && h->plan.key == key) return PLOGP_OK;

    int64_t n_s64 = 0;
    int rc = validate_grid(h, g, &n_s64);
    if (rc != PLOGP_OK) return rc;

    Plan pl;
    pl.key = std::move(key);
    const int n_P = g->P ? g->n_P : (g->P_hi - g->P_lo + 1);
    const int n_m = g->n_m;
    const int n_s = int(n_s64);
    pl.empty = (n_P == 0 || n_m == 0 || g->strategy_mask == 0);
    if (pl.empty) { h->plan = std::move(pl); return PLOGP_OK; }

    const int64_t P_hi = g->P ? g->P[n_P - 1] : g->P_hi;
    pl.n_seg = __builtin_popcount(g->strategy_mask & kSegBits);
    pl.inline_sweep = pl.n_seg == 0 || n_s <= kMaxInlineS;
    // search_mode 1 on tables with non-decreasing gaps.  Long candidate lists: envelope_kernel writes the segmented
    // minima to the scratch rows that fused_kernel reads.  Short lists: the decision kernel prunes its own lists
    // (predictions of short lists keep the exhaustive inline search; the results are the same).
    const bool env_ok = g->search_mode == 1 && pl.n_seg > 0 && n_s > 0 && h->monotone;
    pl.envelope = env_ok && n_s > kMaxInlineS;
    pl.envelope_short = env_ok && n_s <= kMaxInlineS;
    if (pl.envelope) pl.inline_sweep = false;

    // candidates per message size (grid values s <= m)
    std::vector<int32_t> ns_of_m(n_m, 0);
    int ns_max = 0;
    if (pl.n_seg) {
        for (int i = 0; i < n_m; ++i) {
            const uint64_t m = g->m[i];
            int64_t c;
            if (g->s) c = std::upper_bound(g->s, g->s + n_s, m) - g->s;
            else {
                const uint64_t top = std::min<uint64_t>(m, g->s_hi);
                c = (n_s > 0 && top >= g->s_lo) ? int64_t((top - g->s_lo) / g->s_step) + 1 : 0;
            }
            ns_of_m[i] = int32_t(c);
            ns_max = std::max(ns_max, int(c));
        }
    }

    // ---- fused kernel tiling ----
    const int pass_P = kWarps * kFusedR;
    const int total_passes = (n_P + pass_P - 1) / pass_P;
    pl.n_mtiles = (n_m + 31) / 32;
    const long long base_blocks = (long long)pl.n_mtiles * h->T.n_tables;
    const long long target = (long long)h->sm_count * 8;
    int n_ptiles = 1;
    if (base_blocks < target) n_ptiles = int(std::min<long long>(total_passes, (target + base_blocks - 1) / base_blocks));
    n_ptiles = std::min(n_ptiles, 256);
    pl.passes_per_tile = (total_passes + n_ptiles - 1) / n_ptiles;
    pl.n_ptiles = (total_passes + pl.passes_per_tile - 1) / pl.passes_per_tile;
    if (n_P <= 512) { pl.sc_ptiles = 1; pl.sc_passes_per_tile = total_passes; }
    else { pl.sc_ptiles = pl.n_ptiles; pl.sc_passes_per_tile = pl.passes_per_tile; }

    pl.dec_ptiles = (n_P + kDecTileP - 1) / kDecTileP;
    // 16 message sizes per CTA give the widest output rows; small grids trade that for more CTAs
    // (never fewer than one message size per warp)
    pl.dec_mg = kDecMG;
    while (pl.dec_mg > kDecWarps && (long long)((n_m + pl.dec_mg - 1) / pl.dec_mg) * pl.dec_ptiles * h->T.n_tables < (long long)h->sm_count * 4)
        pl.dec_mg >>= 1;
    pl.dec_mgroups = (n_m + pl.dec_mg - 1) / pl.dec_mg;

    // ---- device arrays ----
    std::vector<unsigned char> blob;
    std::vector<uint32_t> m32(n_m);
    for (int i = 0; i < n_m; ++i) m32[i] = uint32_t(g->m[i]);
    const size_t off_m = append_aligned(blob, m32);
    const size_t off_ns = append_aligned(blob, ns_of_m);
    size_t off_P = 0, off_s = 0;
    if (g->P) off_P = append_aligned(blob, std::vector<int32_t>(g->P, g->P + n_P));
    if (pl.n_seg && g->s) {
        std::vector<uint32_t> s32(n_s);
        for (int i = 0; i < n_s; ++i) s32[i] = uint32_t(g->s[i]);
        off_s = append_aligned(blob, s32);
    }

    // Short candidate lists (lane <-> P kernels): Section 2's k for every (m, candidate), as the doubles the kernels multiply with
    const bool short_lists = pl.inline_sweep && pl.n_seg > 0 && n_s > 0;
    if (short_lists) {
        std::vector<double> kt(size_t(n_m) * n_s, 1.0);
        for (int i = 0; i < n_m; ++i) {
            const uint64_t m = g->m[i];
            for (int c = 0; c < ns_of_m[i]; ++c) {
                const uint64_t sv = g->s ? g->s[c] : g->s_lo + uint64_t(c) * g->s_step;
                const uint64_t q = m / sv;
                kt[size_t(i) * n_s + c] = double(q + ((g->k_mode == 0 && q * sv != m) ? 1 : 0));
            }
        }
        pl.off_k = append_aligned(blob, kt);
    }

    // ---- sweep kernel plan: (m, chunk) pairs, heaviest first ----
    if (pl.envelope) {
        // one scratch row per message size
        std::vector<int32_t> pair_base(n_m + 1);
        for (int i = 0; i <= n_m; ++i) pair_base[i] = i;
        pl.n_pairs = n_m;
        pl.off_pair_base = append_aligned(blob, pair_base);
        // short lists: small CTAs; the list of representatives of one message size lives in shared memory
        pl.env_threads = ns_max <= 64 ? 64 : (ns_max <= 4096 ? 256 : 1024);
        pl.env_rep_cap = std::min(std::max(ns_max, 1), 6144);
        pl.env_coarse = std::max(64, (n_P + 1023) / 1024);
        pl.env_max_coarse = (std::max(n_P, 1) - 1 + pl.env_coarse - 1) / pl.env_coarse + 1;
    } else if (!pl.inline_sweep) {
        pl.chunk_len = std::max(2048, ((ns_max + 31) / 32 + kSweepSub - 1) / kSweepSub * kSweepSub);
        std::vector<int32_t> pair_base(n_m + 1, 0);
        struct Pair { int32_t m, chunk, row, len; };
        std::vector<Pair> pairs;
        for (int i = 0; i < n_m; ++i) {
            pair_base[i] = int32_t(pairs.size());
            for (int c = 0; c * pl.chunk_len < ns_of_m[i]; ++c)
                pairs.push_back({i, c, int32_t(pairs.size()), std::min(pl.chunk_len, ns_of_m[i] - c * pl.chunk_len)});
        }
        pair_base[n_m] = int32_t(pairs.size());
        pl.n_pairs = int(pairs.size());
        std::stable_sort(pairs.begin(), pairs.end(), [](const Pair &a, const Pair &b) { return a.len > b.len; });
        std::vector<int32_t> pm(pl.n_pairs), pc(pl.n_pairs), pr(pl.n_pairs);
        for (int i = 0; i < pl.n_pairs; ++i) { pm[i] = pairs[i].m; pc[i] = pairs[i].chunk; pr[i] = pairs[i].row; }
        pl.off_pair_m = append_aligned(blob, pm);
        pl.off_pair_chunk = append_aligned(blob, pc);
        pl.off_pair_row = append_aligned(blob, pr);
        pl.off_pair_base = append_aligned(blob, pair_base);
        pl.sweep_ptiles = (n_P + kThreads * kSweepR - 1) / (kThreads * kSweepR);
    }

    if (blob.size() > h->grid_cap) {
        if (h->d_grid) CK(cudaFree(h->d_grid));
        h->d_grid = nullptr;
        h->grid_cap = 0;
        const size_t cap = std::max<size_t>(blob.size() * 2, 4096);
        CK(cudaMalloc(&h->d_grid, cap));
        h->grid_cap = cap;
    }
    // The source is pageable host memory: the runtime stages it before returning.
    CK(cudaMemcpyAsync(h->d_grid, blob.data(), blob.size(), cudaMemcpyHostToDevice, st));

    GridDev &G = pl.G;
    G.P_list = g->P ? reinterpret_cast<const int32_t *>(h->d_grid + off_P) : nullptr;
    G.n_P = n_P;
    G.P_lo = g->P ? 0 : g->P_lo;
    G.m_list = reinterpret_cast<const uint32_t *>(h->d_grid + off_m);
    G.n_m = n_m;
    G.s_list = (pl.n_seg && g->s) ? reinterpret_cast<const uint32_t *>(h->d_grid + off_s) : nullptr;
    G.n_s = pl.n_seg ? n_s : 0;
    G.s_lo = uint32_t(g->s_lo);
    G.s_step = uint32_t(g->s_step);
    G.ns_of_m = reinterpret_cast<const int32_t *>(h->d_grid + off_ns);
    G.k_list = short_lists ? reinterpret_cast<const double *>(h->d_grid + pl.off_k) : nullptr;
    G.mask = g->strategy_mask;
    G.k_mode = g->k_mode;
    G.lc_max = std::max(1, ceil_log2(P_hi));

    // ---- scratch: sweep partials (per table batch) and Scatter Chain tile prefixes ----
    const bool s1_on = (g->strategy_mask >> 11) & 1u;
    size_t per_table = 0;
    if (!pl.inline_sweep) per_table += size_t(pl.n_seg) * pl.n_pairs * n_P * (sizeof(double) + sizeof(uint32_t)) + 512;
    if (s1_on && pl.n_ptiles > 1) pl.carry_bytes_per_table = size_t(pl.n_ptiles) * (kWarps + 1) * n_m * sizeof(double);
    per_table += pl.carry_bytes_per_table;
    // The gap pre-pass costs a launch: taken where the lane <-> P kernels run many CTAs per table and fill the GPU several times over
    if (pl.inline_sweep && pl.n_seg > 0) {
        const long long ctas_per_table = (long long)pl.dec_mgroups * pl.dec_ptiles;
        pl.use_gaps = ctas_per_table >= 4 && ctas_per_table * h->T.n_tables >= (long long)h->sm_count * 16;
        if (pl.use_gaps) {
            pl.gaps_stride = (1 + n_s + n_m + 1) & ~1;
            pl.gaps_bytes_per_table = size_t(pl.gaps_stride) * sizeof(double);
            per_table += pl.gaps_bytes_per_table;
        }
    }
    pl.tables_per_batch = h->T.n_tables;
    if (!pl.inline_sweep && per_table * h->T.n_tables > kSweepScratchLimit)
        pl.tables_per_batch = int(std::max<size_t>(1, kSweepScratchLimit / per_table));
    pl.tables_per_batch = std::min(pl.tables_per_batch, 65535);
    pl.scratch_bytes = per_table ? per_table * pl.tables_per_batch + 1024 : 0;  // the sections start on 256-byte boundaries
    if (pl.scratch_bytes > h->ws_cap) {
        if (h->d_ws) CK(cudaFree(h->d_ws));
        h->d_ws = nullptr;
        h->ws_cap = 0;
        cudaError_t e = cudaMalloc(&h->d_ws, pl.scratch_bytes);
        if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return PLOGP_E_NOMEM; }
        if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc(scratch)");
        h->ws_cap = pl.scratch_bytes;
    }
    h->plan = std::move(pl);
    return PLOGP_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// plogp_select_best's layout: two planes per table, the ids of Table 1 / Table 2
OutMap default_out_map()
{
    OutMap om{};
    om.planes = 2; om.plane_bcast = 0; om.plane_scat = 1;
    for (int i = 0; i < 16; ++i) om.id_of[i] = uint8_t(i < PLOGP_N_STRATEGIES ? i : 255);
    return om;
}

int run(plogp_tables *h, const plogp_grid *g, bool predict, FusedParams out, cudaStream_t st, int t_begin = 0, int t_end = -1)
{
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev != h->device) return PLOGP_E_INVAL;
    int rc = prepare(h, g, st);
    if (rc != PLOGP_OK) { h->plan = Plan(); return rc; }
    const Plan &pl = h->plan;
    if (pl.empty) return PLOGP_OK;
    const bool s1 = (pl.G.mask >> 11) & 1u;
    // Short candidate lists with segmented strategies: the lane<->P decision kernel; everything else
    // (predictions, long lists reduced by the sweep kernel, Scatter-only grids) goes through fused_kernel.
    const bool use_decide = !predict && pl.inline_sweep && pl.n_seg > 0;
    // the kernel that follows the (optional) Broadcast decision kernel: Scatter strategies only => scatter_kernel
    const bool use_scatter = !predict && ((use_decide ? pl.G.mask & 0x1C00u : pl.G.mask) & 0x3FFu) == 0;
    const int n_ptiles = use_scatter ? pl.sc_ptiles : pl.n_ptiles;
    const int passes_per_tile = use_scatter ? pl.sc_passes_per_tile : pl.passes_per_tile;
    const bool need_carry = s1 && n_ptiles > 1;

    if (t_end < 0) t_end = h->T.n_tables;
    for (int t0 = t_begin; t0 < t_end; t0 += pl.tables_per_batch) {
        const int nt = std::min(pl.tables_per_batch, t_end - t0);
        unsigned char *ws = h->d_ws;
        double *part_time = nullptr;
        uint32_t *part_idx = nullptr;
        double *tile_sum = nullptr;
        if (!pl.inline_sweep) {
            const size_t cells = size_t(nt) * pl.n_seg * pl.n_pairs * pl.G.n_P;
            part_time = reinterpret_cast<double *>(ws);
            ws += align_up(cells * sizeof(double), 256);
            part_idx = reinterpret_cast<uint32_t *>(ws);
            ws += align_up(cells * sizeof(uint32_t), 256);
        }
        if (need_carry) {
            tile_sum = reinterpret_cast<double *>(ws);
            ws += align_up(pl.carry_bytes_per_table * nt, 256);
        }
        double *gaps = nullptr;
        if (pl.use_gaps && pl.inline_sweep && pl.n_seg > 0 && (predict || use_decide)) {
            gaps = reinterpret_cast<double *>(ws);
            GapsParams gp{};
            gp.T = h->T; gp.G = pl.G;
            gp.table0 = t0; gp.n_tables_launch = nt; gp.gaps = gaps; gp.stride = pl.gaps_stride;
            { LaunchTimer lt(h, PLOGP_KERNEL_GAPS, st); CK(launch_gaps(gp, st)); }
            g_launches += 1;
        }

        if (pl.envelope) {
            EnvParams ep{};
            ep.T = h->T; ep.G = pl.G;
            ep.table0 = t0; ep.n_tables_launch = nt;
            ep.part_time = part_time; ep.part_idx = part_idx; ep.n_seg = pl.n_seg;
            ep.rep_cap = pl.env_rep_cap; ep.coarse = pl.env_coarse; ep.max_coarse = pl.env_max_coarse;
            { LaunchTimer lt(h, PLOGP_KERNEL_ENVELOPE, st); CK(launch_envelope(ep, pl.env_threads, st)); }
            g_launches += 1;
        } else if (!pl.inline_sweep && pl.n_pairs > 0) {
            SweepParams sp{};
            sp.T = h->T; sp.G = pl.G;
            sp.pair_m = reinterpret_cast<const int32_t *>(h->d_grid + pl.off_pair_m);
            sp.pair_chunk = reinterpret_cast<const int32_t *>(h->d_grid + pl.off_pair_chunk);
            sp.pair_row = reinterpret_cast<const int32_t *>(h->d_grid + pl.off_pair_row);
            sp.n_pairs = pl.n_pairs; sp.n_ptiles = pl.sweep_ptiles; sp.chunk_len = pl.chunk_len;
            sp.part_time = part_time; sp.part_idx = part_idx; sp.n_seg = pl.n_seg; sp.table0 = t0;
            { LaunchTimer lt(h, PLOGP_KERNEL_SWEEP, st); CK(launch_sweep(sp, nt, st)); }
            g_launches += 1;
        }
        if (need_carry) {
            S1Params s{};
            s.T = h->T; s.G = pl.G;
            s.n_mtiles = pl.n_mtiles; s.n_ptiles = n_ptiles; s.passes_per_tile = passes_per_tile;
            s.table0 = t0; s.n_tables_launch = nt; s.tile_sum = tile_sum;
            { LaunchTimer lt(h, PLOGP_KERNEL_CHAIN_PREFIX, st); CK(launch_s1_tiles(s, st)); }
            g_launches += 1;
        }
        GridDev Gf = pl.G;
        if (predict && pl.inline_sweep && pl.n_seg > 0) {
            // Predictions on short candidate lists: the segmented minima (planes 2, 5, 9 and the best segment sizes)
            // come from the lane<->P kernel; fused_kernel then writes the closed-form planes only.
            SegminParams sp{};
            sp.T = h->T; sp.G = pl.G;
            sp.n_mgroups = (pl.G.n_m + kSegMG - 1) / kSegMG; sp.n_ptiles = (pl.G.n_P + kSegTileP - 1) / kSegTileP;
            sp.table0 = t0; sp.n_tables_launch = nt; sp.out_table0 = out.out_table0;
            sp.p_time = out.p_time; sp.p_best_s = out.p_best_s;
            sp.gaps = gaps; sp.gaps_stride = pl.gaps_stride;
            sp.vec_out = (pl.G.n_m % 2 == 0) && reinterpret_cast<uintptr_t>(out.p_time) % 16 == 0 &&
                         (!out.p_best_s || reinterpret_cast<uintptr_t>(out.p_best_s) % 8 == 0);
            { LaunchTimer lt(h, PLOGP_KERNEL_SEGMIN, st); CK(launch_segmin(sp, st)); }
            g_launches += 1;
            Gf.mask &= ~kSegBits;
            Gf.n_s = 0;
            if (!Gf.mask) continue;
        }
        if (use_decide) {
            // Broadcast half with lanes <-> P; the Scatter half (no candidate lists) follows in fused_kernel.
            DecideParams dp{};
            dp.T = h->T; dp.G = pl.G;
            dp.G.mask &= 0x3FFu;
            dp.n_mgroups = pl.dec_mgroups; dp.n_ptiles = pl.dec_ptiles; dp.mg = pl.dec_mg;
            dp.table0 = t0; dp.n_tables_launch = nt; dp.out_table0 = out.out_table0; dp.om = out.om;
            dp.d_strategy = out.d_strategy; dp.d_sbytes = out.d_sbytes; dp.d_time = out.d_time;
            dp.envelope = pl.envelope_short ? 1 : 0;
            dp.gaps = gaps; dp.gaps_stride = pl.gaps_stride;
            dp.vec_out = (pl.G.n_m % 2 == 0) && pl.dec_mg >= 2 && reinterpret_cast<uintptr_t>(out.d_time) % 16 == 0 &&
                         reinterpret_cast<uintptr_t>(out.d_sbytes) % 8 == 0 && reinterpret_cast<uintptr_t>(out.d_strategy) % 2 == 0;
            { LaunchTimer lt(h, PLOGP_KERNEL_DECIDE, st); CK(launch_decide(dp, st)); }
            g_launches += 1;
            Gf.mask &= 0x1C00u;
            Gf.n_s = 0;
            if (!Gf.mask) continue;
        }
        FusedParams fp = out;
        fp.T = h->T; fp.G = Gf;
        fp.n_mtiles = pl.n_mtiles; fp.n_ptiles = n_ptiles; fp.passes_per_tile = passes_per_tile;
        fp.table0 = t0; fp.n_tables_launch = nt;
        fp.s1_sums = tile_sum;
        // part_time doubles as the "segmented minima come from the sweep kernel" switch
        fp.part_time = pl.inline_sweep ? nullptr : part_time;
        fp.part_idx = part_idx;
        fp.pair_base = pl.inline_sweep ? nullptr : reinterpret_cast<const int32_t *>(h->d_grid + pl.off_pair_base);
        fp.n_pairs = pl.n_pairs; fp.n_seg = pl.n_seg;
        if (use_scatter) { LaunchTimer lt(h, PLOGP_KERNEL_SCATTER, st); CK(launch_scatter(fp, st)); }
        else { LaunchTimer lt(h, PLOGP_KERNEL_FUSED, st); CK(launch_fused(fp, predict, st)); }
        g_launches += 1;
    }
    return PLOGP_OK;
}

}  // namespace

extern "C" {

// Validates host tables and lays them out as the kernels read them (key | gap | slope, padded).
static int build_tables(int n_tables, int n_bp, int npad, const uint64_t *sizes_bytes, int sizes_shared,
                        const double *gap, const double *latency, std::vector<double> &tab, std::vector<double> &lat,
                        bool *monotone)
{
    *monotone = true;
    try {
        tab.assign(size_t(n_tables) * 3 * npad, 0.0);
        lat.assign(latency, latency + n_tables);
    } catch (const std::bad_alloc &) { return PLOGP_E_NOMEM; }

    const double inf = std::numeric_limits<double>::infinity();
    for (int t = 0; t < n_tables; ++t) {
        const uint64_t *sz = sizes_bytes + (sizes_shared ? 0 : size_t(t) * n_bp);
        const double *gp = gap + size_t(t) * n_bp;
        if (!std::isfinite(lat[t]) || lat[t] < 0.0) return PLOGP_E_INVAL;
        for (int i = 0; i < n_bp; ++i) {
            if (!std::isfinite(gp[i]) || gp[i] < 0.0) return PLOGP_E_INVAL;
            if (i && sz[i] <= sz[i - 1]) return PLOGP_E_INVAL;
            if (i && gp[i] < gp[i - 1]) *monotone = false;
            if (double(sz[i]) >= kTwo53) return PLOGP_E_RANGE;
        }
        // Above the last size the last interval's line is continued: a falling line would turn g negative for
        // large arguments, and the kernels compare times through their (sign-free) high words.
        if (gp[n_bp - 1] < gp[n_bp - 2]) return PLOGP_E_RANGE;
        double *key = tab.data() + size_t(t) * 3 * npad, *g0 = key + npad, *sl = g0 + npad;
        for (int i = 0; i < npad; ++i) {
            if (i <= n_bp - 2) {
                key[i] = double(sz[i]);
                g0[i] = gp[i];
                sl[i] = (gp[i + 1] - gp[i]) / double(sz[i + 1] - sz[i]);
            } else {
                key[i] = inf;
                g0[i] = 0.0;
                sl[i] = 0.0;
            }
        }
    }
    return PLOGP_OK;
}

int plogp_table_load(int n_tables, int n_bp, const uint64_t *sizes_bytes, int sizes_shared,
                     const double *gap, const double *latency, plogp_tables **out)
{
    if (!sizes_bytes || !gap || !latency || !out) return PLOGP_E_INVAL;
    if (n_tables < 1 || n_bp < 2) return PLOGP_E_INVAL;
    if (n_bp > PLOGP_MAX_BREAKPOINTS) return PLOGP_E_RANGE;
    int npad = 2;
    while (npad < n_bp) npad <<= 1;  // >= n_bp: at least one +inf key follows the last interval

    std::vector<double> tab, lat;
    bool monotone = false;
    const int brc = build_tables(n_tables, n_bp, npad, sizes_bytes, sizes_shared, gap, latency, tab, lat, &monotone);
    if (brc != PLOGP_OK) return brc;

    plogp_tables *h = new (std::nothrow) plogp_tables();
    if (!h) return PLOGP_E_NOMEM;
    auto fail = [&](int rc) { plogp_table_free(h); return rc; };
    cudaError_t e;
    if ((e = cudaGetDevice(&h->device)) != cudaSuccess) return fail(cuda_fail(e, "cudaGetDevice"));
    if ((e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device)) != cudaSuccess)
        return fail(cuda_fail(e, "cudaDeviceGetAttribute"));
    if ((e = cudaMalloc(&h->d_tab, tab.size() * sizeof(double))) != cudaSuccess)
        return fail(e == cudaErrorMemoryAllocation ? (cudaGetLastError(), PLOGP_E_NOMEM) : cuda_fail(e, "cudaMalloc(tables)"));
    if ((e = cudaMalloc(&h->d_lat, lat.size() * sizeof(double))) != cudaSuccess)
        return fail(e == cudaErrorMemoryAllocation ? (cudaGetLastError(), PLOGP_E_NOMEM) : cuda_fail(e, "cudaMalloc(latency)"));
    if ((e = cudaMemcpy(h->d_tab, tab.data(), tab.size() * sizeof(double), cudaMemcpyHostToDevice)) != cudaSuccess)
        return fail(cuda_fail(e, "cudaMemcpy(tables)"));
    if ((e = cudaMemcpy(h->d_lat, lat.data(), lat.size() * sizeof(double), cudaMemcpyHostToDevice)) != cudaSuccess)
        return fail(cuda_fail(e, "cudaMemcpy(latency)"));
    h->T.tab = h->d_tab;
    h->T.lat = h->d_lat;
    h->T.n_tables = n_tables;
    h->T.n_bp = n_bp;
    h->T.npad = npad;
    h->monotone = monotone;
    *out = h;
    return PLOGP_OK;
}

int plogp_table_update(plogp_tables *h, const uint64_t *sizes_bytes, int sizes_shared, const double *gap,
                       const double *latency, void *stream)
{
    if (!h || !sizes_bytes || !gap || !latency) return PLOGP_E_INVAL;
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev != h->device) return PLOGP_E_INVAL;
    std::vector<double> tab, lat;
    bool monotone = false;
    const int brc = build_tables(h->T.n_tables, h->T.n_bp, h->T.npad, sizes_bytes, sizes_shared, gap, latency, tab, lat, &monotone);
    if (brc != PLOGP_OK) return brc;  // the tables on the device are untouched
    h->monotone = monotone;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // pageable sources: the runtime stages them before returning, so the vectors may go out of scope
    CK(cudaMemcpyAsync(h->d_tab, tab.data(), tab.size() * sizeof(double), cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(h->d_lat, lat.data(), lat.size() * sizeof(double), cudaMemcpyHostToDevice, st));
    return PLOGP_OK;
}

int plogp_table_free(plogp_tables *h)
{
    if (!h) return PLOGP_OK;
    int rc = PLOGP_OK;
    void *bufs[] = {h->d_tab, h->d_lat, h->d_grid, h->d_ws, h->d_stage[0], h->d_stage[1]};
    for (int i = 0; i < 2; ++i) {
        if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
        if (h->ev_copied[i]) cudaEventDestroy(h->ev_copied[i]);
    }
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    for (void *b : bufs) {
        if (b) {
            cudaError_t e = cudaFree(b);
            if (e != cudaSuccess) rc = cuda_fail(e, "cudaFree");
        }
    }
    for (auto &t : h->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
    delete h;
    return rc;
}

int plogp_profile_enable(plogp_tables *h, int enable)
{
    if (!h) return PLOGP_E_INVAL;
    h->profiling = enable != 0;
    return PLOGP_OK;
}

int plogp_profile_read(plogp_tables *h, double *ms, int32_t *launches)
{
    if (!h || !ms || !launches) return PLOGP_E_INVAL;
    for (int k = 0; k < PLOGP_N_KERNEL_KINDS; ++k) { ms[k] = 0.0; launches[k] = 0; }
    int rc = PLOGP_OK;
    for (auto &t : h->timed) {
        float v = 0.f;
        cudaError_t e = cudaEventSynchronize(t.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&v, t.a, t.b);
        if (e == cudaSuccess) { ms[t.kind] += v; launches[t.kind] += 1; }
        else rc = cuda_fail(e, "cudaEventElapsedTime");
        cudaEventDestroy(t.a);
        cudaEventDestroy(t.b);
    }
    h->timed.clear();
    return rc;
}

int plogp_predict(plogp_tables *tables, const plogp_grid *grid, double *d_time, uint32_t *d_best_s, void *stream)
{
    if (!tables || !grid || !d_time) return PLOGP_E_INVAL;
    FusedParams out{};
    out.om = default_out_map();
    out.p_time = d_time;
    out.p_best_s = d_best_s;
    return run(tables, grid, true, out, static_cast<cudaStream_t>(stream));
}

int plogp_select_best(plogp_tables *tables, const plogp_grid *grid, uint8_t *d_strategy, uint32_t *d_s_bytes,
                      double *d_time, void *stream)
{
    if (!tables || !grid || !d_strategy || !d_s_bytes || !d_time) return PLOGP_E_INVAL;
    FusedParams out{};
    out.om = default_out_map();
    out.d_strategy = d_strategy;
    out.d_sbytes = d_s_bytes;
    out.d_time = d_time;
    return run(tables, grid, false, out, static_cast<cudaStream_t>(stream));
}

int plogp_select_best_host(plogp_tables *h, const plogp_grid *grid, uint8_t *h_strategy, uint32_t *h_s_bytes,
                           double *h_time, void *stream)
{
    if (!h || !grid || !h_strategy || !h_s_bytes || !h_time) return PLOGP_E_INVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev != h->device) return PLOGP_E_INVAL;
    int rc = prepare(h, grid, st);
    if (rc != PLOGP_OK) { h->plan = Plan(); return rc; }
    if (h->plan.empty) return PLOGP_OK;
    const size_t cells = size_t(2) * h->plan.G.n_P * h->plan.G.n_m;  // per table
    const size_t per_table = cells * 13 + 3 * 256;
    // tables per staging set: at most 512 MiB, at least one table
    const int batch = int(std::min<size_t>(h->T.n_tables, std::max<size_t>(1, (size_t(512) << 20) / per_table)));
    const size_t need = per_table * batch;
    if (need > h->stage_cap) {
        for (int i = 0; i < 2; ++i) {
            if (h->d_stage[i]) CK(cudaFree(h->d_stage[i]));
            h->d_stage[i] = nullptr;
        }
        h->stage_cap = 0;
        for (int i = 0; i < 2; ++i) {
            cudaError_t e = cudaMalloc(&h->d_stage[i], need);
            if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return PLOGP_E_NOMEM; }
            if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc(staging)");
        }
        h->stage_cap = need;
    }
    if (!h->copy_stream) {
        CK(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CK(cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming));
            CK(cudaEventCreateWithFlags(&h->ev_copied[i], cudaEventDisableTiming));
        }
    }
    auto align = [](size_t x) { return (x + 255) / 256 * 256; };
    int slot = 0;
    for (int t0 = 0; t0 < h->T.n_tables; t0 += batch, slot ^= 1) {
        const int nt = std::min(batch, h->T.n_tables - t0);
        // layout of a staging set: time | segment size | strategy, each for nt tables
        double *s_time = reinterpret_cast<double *>(h->d_stage[slot]);
        uint32_t *s_sb = reinterpret_cast<uint32_t *>(h->d_stage[slot] + align(cells * 8 * batch));
        uint8_t *s_id = h->d_stage[slot] + align(cells * 8 * batch) + align(cells * 4 * batch);
        if (t0 >= 2 * batch) {  // the set's previous copy has left
            cudaError_t ew = cudaStreamWaitEvent(st, h->ev_copied[slot], 0);
            if (ew != cudaSuccess) { rc = cuda_fail(ew, "cudaStreamWaitEvent"); break; }
        }
        FusedParams out{};
        out.om = default_out_map();
        out.d_time = s_time;
        out.d_sbytes = s_sb;
        out.d_strategy = s_id;
        out.out_table0 = t0;  // the staging set holds tables t0 .. t0 + nt - 1
        rc = run(h, grid, false, out, st, t0, t0 + nt);
        // On any failure the loop ends here, and both streams are drained below before the call returns: no
        // copy into the caller's arrays is left in flight.
        cudaError_t e = cudaSuccess;
        if (rc == PLOGP_OK) e = cudaEventRecord(h->ev_done[slot], st);
        if (rc == PLOGP_OK && e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_stream, h->ev_done[slot], 0);
        if (rc == PLOGP_OK && e == cudaSuccess)
            e = cudaMemcpyAsync(h_time + size_t(t0) * cells, s_time, cells * 8 * nt, cudaMemcpyDeviceToHost, h->copy_stream);
        if (rc == PLOGP_OK && e == cudaSuccess)
            e = cudaMemcpyAsync(h_s_bytes + size_t(t0) * cells, s_sb, cells * 4 * nt, cudaMemcpyDeviceToHost, h->copy_stream);
        if (rc == PLOGP_OK && e == cudaSuccess)
            e = cudaMemcpyAsync(h_strategy + size_t(t0) * cells, s_id, cells * nt, cudaMemcpyDeviceToHost, h->copy_stream);
        if (rc == PLOGP_OK && e == cudaSuccess) e = cudaEventRecord(h->ev_copied[slot], h->copy_stream);
        if (rc == PLOGP_OK && e != cudaSuccess) rc = cuda_fail(e, "plogp_select_best_host: copy pipeline");
        if (rc != PLOGP_OK) break;
    }
    cudaError_t e1 = cudaStreamSynchronize(h->copy_stream), e2 = cudaStreamSynchronize(st);
    if (rc != PLOGP_OK) { cudaGetLastError(); return rc; }
    if (e1 != cudaSuccess) return cuda_fail(e1, "cudaStreamSynchronize(copy)");
    if (e2 != cudaSuccess) return cuda_fail(e2, "cudaStreamSynchronize");
    return PLOGP_OK;
}

int plogp_select_best_collective(plogp_tables *h, const plogp_grid *grid, int collective, uint8_t *d_strategy,
                                 uint32_t *d_s_bytes, double *d_time, void *stream)
{
    if (!h || !grid || !d_strategy || !d_s_bytes || !d_time) return PLOGP_E_INVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    plogp_grid g = *grid;
    FusedParams out{};
    out.om = default_out_map();
    out.om.planes = 1; out.om.plane_bcast = 0; out.om.plane_scat = 0;
    out.d_strategy = d_strategy; out.d_sbytes = d_s_bytes; out.d_time = d_time;
    switch (collective) {
    case PLOGP_GATHER:  // the Scatter strategies run backwards: ids 10, 11, 12 -> 13, 14, 15
        g.strategy_mask &= 0x1C00u;
        for (int i = 10; i <= 12; ++i) out.om.id_of[i] = uint8_t(i + 3);
        return run(h, &g, false, out, st);
    case PLOGP_REDUCE: {  // the Broadcast strategies without a handshake run backwards: 0 2 3 5 6 7 9 -> 16 .. 22
        g.strategy_mask &= 0x2EDu;
        static const int from[7] = {0, 2, 3, 5, 6, 7, 9};
        for (int i = 0; i < 7; ++i) out.om.id_of[from[i]] = uint8_t(16 + i);
        return run(h, &g, false, out, st);
    }
    case PLOGP_BARRIER: {  // one decision per (table, P); the message sizes play no part
        g.strategy_mask &= 0xC9u;
        int dev = 0;
        CK(cudaGetDevice(&dev));
        if (dev != h->device) return PLOGP_E_INVAL;
        int rc = prepare(h, &g, st);
        if (rc != PLOGP_OK) { h->plan = Plan(); return rc; }
        if (h->plan.empty) return PLOGP_OK;  // no process count, no message size to carry the plan, or no strategy
        CK(launch_barrier(h->T, h->plan.G, 0, h->T.n_tables, d_strategy, d_s_bytes, d_time, st));
        g_launches += 1;
        return PLOGP_OK;
    }
    default:
        return PLOGP_E_INVAL;
    }
}

int plogp_segment_surface(plogp_tables *h, const plogp_grid *grid, double *d_surface, void *stream)
{
    if (!h || !grid || !d_surface) return PLOGP_E_INVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev != h->device) return PLOGP_E_INVAL;
    int rc = prepare(h, grid, st);
    if (rc != PLOGP_OK) { h->plan = Plan(); return rc; }
    const Plan &pl = h->plan;
    if (pl.empty || pl.n_seg == 0 || pl.G.n_s == 0) return PLOGP_OK;
    for (int t0 = 0; t0 < h->T.n_tables; t0 += 65535) {
        SensParams sp{};
        sp.T = h->T; sp.G = pl.G;
        sp.table0 = t0; sp.n_tables_launch = std::min(65535, h->T.n_tables - t0); sp.out_table0 = 0;
        sp.surface = d_surface;
        CK(launch_surface(sp, st));
        g_launches += 1;
    }
    return PLOGP_OK;
}

int plogp_segment_sensitivity(plogp_tables *h, const plogp_grid *grid, uint64_t s_fixed, const double *d_pred_time,
                              double *d_time_fixed, double *d_ratio, void *stream)
{
    if (!h || !grid || !d_time_fixed) return PLOGP_E_INVAL;
    if ((d_ratio == nullptr) != (d_pred_time == nullptr)) return PLOGP_E_INVAL;
    if (s_fixed == 0 || grid->dtype_bytes == 0 || s_fixed % grid->dtype_bytes) return PLOGP_E_INVAL;
    if (s_fixed >= kTwo32) return PLOGP_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev != h->device) return PLOGP_E_INVAL;
    int rc = prepare(h, grid, st);
    if (rc != PLOGP_OK) { h->plan = Plan(); return rc; }
    const Plan &pl = h->plan;
    if (pl.empty || pl.n_seg == 0) return PLOGP_OK;
    // enough CTAs to fill the GPU, each with a run of process counts per warp
    const long long base_blocks = (long long)((pl.G.n_m + 31) / 32) * h->T.n_tables;
    int p_per_cta = pl.G.n_P;
    while (p_per_cta > 8 && base_blocks * ((pl.G.n_P + p_per_cta - 1) / p_per_cta) < (long long)h->sm_count * 8) p_per_cta = (p_per_cta + 1) / 2;
    for (int t0 = 0; t0 < h->T.n_tables; t0 += 65535) {
        SensParams sp{};
        sp.T = h->T; sp.G = pl.G;
        sp.table0 = t0; sp.n_tables_launch = std::min(65535, h->T.n_tables - t0); sp.out_table0 = 0;
        sp.s_fixed = uint32_t(s_fixed); sp.p_per_cta = p_per_cta;
        sp.pred_time = d_pred_time; sp.time_fixed = d_time_fixed; sp.ratio = d_ratio;
        CK(launch_fixed(sp, st));
        g_launches += 1;
    }
    return PLOGP_OK;
}

int plogp_decision_boundaries(int n_tables, int n_P, int n_m, const uint8_t *d_strategy, uint8_t *d_boundary, void *stream)
{
    if (n_tables < 0 || n_P < 0 || n_m < 0) return PLOGP_E_INVAL;
    if (n_tables == 0 || n_P == 0 || n_m == 0) return PLOGP_OK;
    if (!d_strategy || !d_boundary) return PLOGP_E_INVAL;
    int dev = 0, sms = 0;
    CK(cudaGetDevice(&dev));
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CK(launch_boundaries(d_strategy, d_boundary, 2LL * n_tables, n_P, n_m, sms, static_cast<cudaStream_t>(stream)));
    g_launches += 1;
    return PLOGP_OK;
}

const char *plogp_status_string(int status)
{
    switch (status) {
    case PLOGP_OK: return "ok";
    case PLOGP_E_INVAL: return "invalid argument";
    case PLOGP_E_NOMEM: return "out of memory";
    case PLOGP_E_CUDA: return "CUDA runtime error";
    case PLOGP_E_RANGE: return "value out of the supported range";
    default: return "unknown status";
    }
}

const char *plogp_last_cuda_error(void) { return g_cuda_error.c_str(); }

uint64_t plogp_kernel_launches(void) { return g_launches.load(); }

double plogp_fp64_fma_rate(double milliseconds)
{
    if (!(milliseconds > 0.0)) return double(PLOGP_E_INVAL);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return double(PLOGP_E_CUDA);
    double *sink = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    double rate = double(PLOGP_E_CUDA);
    const int blocks = sms * 4;
    const double fma_per_iter = double(blocks) * kThreads * 32.0;
    do {
        if (cudaMalloc(&sink, sizeof(double)) != cudaSuccess) break;
        if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) break;
        int iters = 2000;
        float ms = 0.f;
        bool ok = true;
        for (int round = 0; round < 3 && ok; ++round) {  // warm-up, calibration, measurement
            ok = cudaEventRecord(e0) == cudaSuccess && launch_fp64_probe(sink, iters, blocks, nullptr) == cudaSuccess &&
                 (g_launches += 1, true) &&
                 cudaEventRecord(e1) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess &&
                 cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess;
            if (ok && round == 1 && ms > 0.f) iters = int(std::min(2e8, std::max(2000.0, iters * milliseconds / ms)));
        }
        if (ok && ms > 0.f) rate = fma_per_iter * iters / (ms * 1e-3);
    } while (0);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (sink) cudaFree(sink);
    return rate;
}

}  // extern "C"
