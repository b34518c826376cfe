/*
 * plogp.h — C ABI of the pLogP collective-communication tuner for one NVIDIA B200 (sm_100a).
 *
 * The library evaluates, on the GPU, the completion-time models that "Fast Tuning of
 * Intra-Cluster Collective Communications" (Barchet-Estefanel & Mounié) prints for the
 * Broadcast strategies (Table 1) and the Scatter strategies (Table 2), searches the segment
 * size that minimises each segmented model (Section 3.1) and selects, for every parameter set
 * (communication pattern, message size, number of processes — Section 1), the strategy with the
 * lowest predicted time (Sections 1 and 5).  The network enters through the pLogP parameters
 * of Section 2: the latency L and the gap g(m), measured at a list of message sizes.
 *
 * All arithmetic is IEEE double.  There is no CPU fallback: every call needs a CUDA device of
 * compute capability 10.0.
 *
 * Strategy ids (Table 1 rows in print order, then Table 2 rows):
 *    0 Flat Tree                  (P-1) g(m) + L
 *    1 Flat Tree Rendezvous       (P-1) g(m) + 2 g(1) + 3 L
 *    2 Segmented Flat Tree        (P-1) (g(s) k) + L
 *    3 Chain                      (P-1) (g(m) + L)
 *    4 Chain Rendezvous           (P-1) (g(m) + 2 g(1) + 3 L)
 *    5 Segmented Chain (Pipeline) (P-1) (g(s) + L) + g(s) (k-1)
 *    6 Binary Tree                ceil(log2 P) (2 g(m) + L)      (printed as an upper bound)
 *    7 Binomial Tree              floor(log2 P) g(m) + ceil(log2 P) L
 *    8 Binomial Tree Rendezvous   floor(log2 P) g(m) + ceil(log2 P) (2 g(1) + 3 L)
 *    9 Segmented Binomial Tree    floor(log2 P) g(s) k + ceil(log2 P) L
 *   10 Scatter Flat Tree          (P-1) g(m) + L
 *   11 Scatter Chain              sum_{j=1..P-1} g(j m) + (P-1) L
 *   12 Scatter Binomial Tree      sum_{j=0..ceil(log2 P)-1} g(2^j m) + ceil(log2 P) L
 *
 * Conventions the paper leaves open (fixed here, identical in every entry point):
 *   - g(x) is linear in x (bytes) between neighbouring measured sizes; below the first size it
 *     keeps the first value; above the last size the last interval's line is continued.
 *   - k, the number of segments of Section 2, is ceil(m/s) (k_mode 0) or floor(m/s) as Section
 *     3.1 prints it (k_mode 1); every segment costs g(s).
 *   - candidate segment sizes for a message m are the grid values s <= m; if none fits, the
 *     message is sent whole (s = m, k = 1) and best_s reports m.
 *   - ties: the smallest segment size, then the lowest strategy id.  (With search_mode 1 two segment sizes of
 *     ids 2 / 9 whose g(s) k differ but whose predicted times round to the same double may resolve to either.)
 *
 * Threading: calls on one plogp_tables handle must not overlap in time on the host, and their
 * device work must be ordered (use one stream, or order the streams yourself): a handle owns
 * device scratch that its calls reuse.  Different handles are independent.
 */
#ifndef PLOGP_H
#define PLOGP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PLOGP_N_STRATEGIES 13
#define PLOGP_N_SEGMENTED 3      /* ids 2, 5, 9, in this order in best_s outputs */
#define PLOGP_MAX_BREAKPOINTS 1024
#define PLOGP_MAX_INLINE_S 64    /* informational: longer segment lists go through the sweep kernel */

typedef enum {
    PLOGP_OK = 0,
    PLOGP_E_INVAL = -1, /* malformed argument (null pointer, n_bp < 2, sizes not increasing, NaN or negative
                           gap, P < 2, m or s not a positive multiple of dtype_bytes, lists not ascending) */
    PLOGP_E_NOMEM = -2, /* host or device allocation failed */
    PLOGP_E_CUDA = -3,  /* a CUDA runtime call failed; plogp_last_cuda_error() names it */
    PLOGP_E_RANGE = -4  /* m, s or a table size too large: m and s must be < 2^32, sizes < 2^53,
                           n_bp <= PLOGP_MAX_BREAKPOINTS, P <= 2^30, P_hi * m < 2^53 (so that j * m is exact in a
                           double); or a table whose last gap is below the one before it (continued above the
                           table, that line would make g negative) */
} plogp_status;

/* Opaque set of pLogP parameter tables resident on the current CUDA device. */
typedef struct plogp_tables plogp_tables;

/*
 * Upload n_tables independent pLogP parameter sets (Section 2: gap g at n_bp message sizes and
 * the latency L of each network).
 *   sizes_bytes  HOST, [n_bp] when sizes_shared != 0, else [n_tables][n_bp]; strictly increasing.
 *   gap          HOST, [n_tables][n_bp]; finite, >= 0; any time unit (the outputs use the same).  The last
 *                gap must not be below the one before it (PLOGP_E_RANGE): all predicted times are then >= 0.
 *   latency      HOST, [n_tables]; finite, >= 0.
 *   out          receives the handle; release it with plogp_table_free.
 * The host arrays are copied before the call returns; the caller keeps them.  The call
 * synchronises with the device (it allocates).  Nothing is written to *out on error.
 */
int plogp_table_load(int n_tables, int n_bp, const uint64_t *sizes_bytes, int sizes_shared,
                     const double *gap, const double *latency, plogp_tables **out);

/*
 * Replace the contents of every table of a handle (same n_tables and n_bp as at plogp_table_load; same
 * argument meaning and checks) without reallocating anything: for callers that re-tune the same grid as the
 * measured pLogP parameters of Section 2 change.  The host arrays are copied before the call returns; the
 * device copy is enqueued on `stream`, ordered before later calls on that stream.  On an error the tables on the
 * device are unchanged.
 */
int plogp_table_update(plogp_tables *tables, const uint64_t *sizes_bytes, int sizes_shared,
                       const double *gap, const double *latency, void *stream);

/* Release a handle and its device memory (synchronises). NULL is accepted. */
int plogp_table_free(plogp_tables *tables);

/*
 * The parameter sets to evaluate: process counts P, message sizes m (Section 1's "message size,
 * number of processes") and candidate segment sizes s (Section 2: a multiple of the basic
 * datatype's size).  All arrays are HOST memory and are copied by the call.
 */
typedef struct {
    const int32_t *P;   /* [n_P] ascending, each >= 2; or NULL for the contiguous range P_lo..P_hi */
    int32_t n_P;        /* ignored when P == NULL */
    int32_t P_lo, P_hi; /* used when P == NULL; 2 <= P_lo <= P_hi */
    const uint64_t *m;  /* [n_m] bytes, ascending, positive multiples of dtype_bytes */
    int32_t n_m;
    const uint64_t *s;  /* [n_s] bytes, ascending, positive multiples of dtype_bytes; or NULL for
                           every s_lo + i * s_step <= s_hi */
    int64_t n_s;        /* ignored when s == NULL */
    uint64_t s_lo, s_hi, s_step;
    uint32_t dtype_bytes;   /* size of the basic datatype, > 0 */
    uint32_t strategy_mask; /* bit i enables strategy id i */
    int32_t k_mode;         /* 0: k = ceil(m/s); 1: k = floor(m/s) */
    int32_t search_mode;    /* how the minimum over s of Section 3.1 is found; the results are the same:
                               0: exhaustive, every (P, m, s) cell is evaluated (the default);
                               1: lower envelope: ids 2 and 9 take the s with the smallest g(s) k once per m, id 5
                                  walks the lower envelope of its lines in P (only for tables whose gaps never
                                  decrease with the size; other tables silently take the exhaustive search) */
} plogp_grid;

/*
 * Evaluate every enabled model of Table 1 / Table 2 on the grid; the segmented ones (ids 2, 5,
 * 9) are reduced over the candidate segment sizes as Section 3.1 describes.
 *   d_time    DEVICE, [n_tables][13][n_P][n_m] doubles, m fastest; planes of disabled strategies
 *             are left untouched.
 *   d_best_s  DEVICE, [n_tables][3][n_P][n_m] uint32 bytes for ids 2, 5, 9 (disabled: untouched);
 *             may be NULL.
 *   stream    a cudaStream_t (NULL = default stream).  Work is enqueued; the call does not wait
 *             for it, but may synchronise when the handle's scratch has to grow.
 * Both outputs belong to the caller.
 * The handle keeps the launch plan of the last grid: a call with the same grid (and per-kernel
 * timing off) copies nothing and allocates nothing, it only launches kernels on `stream`, so a
 * loop of such calls may be captured into a CUDA graph and replayed.  The first call with a new
 * grid uploads the grid and may allocate scratch: make it outside the capture.
 */
int plogp_predict(plogp_tables *tables, const plogp_grid *grid, double *d_time, uint32_t *d_best_s,
                  void *stream);

/*
 * Decision table (Sections 1 and 5): for every table, collective (0 = Broadcast, ids 0..9;
 * 1 = Scatter, ids 10..12), P and m, the enabled strategy with the lowest predicted time.
 *   d_strategy  DEVICE, uint8  [n_tables][2][n_P][n_m], the winning id
 *   d_s_bytes   DEVICE, uint32 [n_tables][2][n_P][n_m], its segment size, 0 when unsegmented
 *   d_time      DEVICE, double [n_tables][2][n_P][n_m], its predicted time
 * A collective with no enabled strategy leaves its planes untouched.  Same stream and ownership
 * rules as plogp_predict.
 */
int plogp_select_best(plogp_tables *tables, const plogp_grid *grid, uint8_t *d_strategy,
                      uint32_t *d_s_bytes, double *d_time, void *stream);

/*
 * Decision tables for the collectives that Section 3 names as built "in a very similar way" as Broadcast and Scatter
 * — Gather, Reduce, Barrier — but for which the paper prints no models.  The models used here are derived (the
 * paper has no counterpart to cite for the formulas themselves): with the gap charged to a node's port for receives
 * as for sends, a Gather is a Scatter run backwards in time and a Reduce a Broadcast run backwards (communication
 * only: pLogP has no parameter for the combine operation), so each takes the mirrored strategy's time; a Barrier is a
 * Reduce followed by a Broadcast of one-byte messages.
 *   collective   PLOGP_GATHER:  ids 13 Flat Tree, 14 Chain, 15 Binomial Tree              (mirrors of ids 10, 11, 12)
 *                PLOGP_REDUCE:  ids 16 Flat, 17 Segmented Flat, 18 Chain, 19 Segmented Chain, 20 Binary, 21 Binomial,
 *                               22 Segmented Binomial Tree                                (mirrors of ids 0 2 3 5 6 7 9)
 *                PLOGP_BARRIER: ids 23 Flat Tree 2((P-1) g(1) + L), 24 Chain 2 (P-1)(g(1) + L),
 *                               25 Binary Tree 2 ceil(log2 P)(2 g(1) + L), 26 Binomial Tree 2 (floor(log2 P) g(1) + ceil(log2 P) L)
 *   grid->strategy_mask  bit i enables the strategy that mirrors printed id i (Barrier: the tree shape of ids 0, 3, 6, 7);
 *                other bits are ignored.  All other grid fields as in plogp_select_best.
 *   d_strategy / d_s_bytes / d_time   DEVICE, one plane per table: [n_tables][n_P][n_m]; for PLOGP_BARRIER
 *                [n_tables][n_P] (the message sizes play no part, but the grid must still carry at least one).
 * A collective with no enabled strategy leaves its outputs untouched.  Same stream and ownership rules as
 * plogp_select_best; Gather and Reduce run the same kernels.
 */
enum { PLOGP_GATHER = 2, PLOGP_REDUCE = 3, PLOGP_BARRIER = 4 };
int plogp_select_best_collective(plogp_tables *tables, const plogp_grid *grid, int collective, uint8_t *d_strategy,
                                 uint32_t *d_s_bytes, double *d_time, void *stream);

/*
 * plogp_select_best with HOST outputs: the same decision table (Sections 1 and 5), delivered into the
 * caller's host arrays h_strategy / h_s_bytes / h_time, each [n_tables][2][n_P][n_m].  The tables are
 * processed in batches through two device staging sets owned by the handle (at most 512 MiB each, or one
 * table), so the device never holds the whole decision table, and the device-to-host copy of one batch runs
 * while the next batch is computed.  Page-locked host arrays are needed for that overlap (pageable ones work,
 * more slowly).  Planes of a collective with no enabled strategy are copied from staging unchanged, i.e. their
 * contents are unspecified.  The call returns after the last byte has arrived (it synchronises `stream` and
 * its own copy stream); it may allocate staging memory on first use.
 */
int plogp_select_best_host(plogp_tables *tables, const plogp_grid *grid, uint8_t *h_strategy,
                           uint32_t *h_s_bytes, double *h_time, void *stream);

/*
 * Model surface over the segment size (Section 3.1 searches the s that minimises these values): the models of the
 * segmented strategies (ids 2, 5, 9 of Table 1, in this order) for every candidate s of the grid.
 *   d_surface  DEVICE, double [n_tables][3][n_P][n_m][n_s], s fastest, n_s = number of candidates of the grid;
 *              NaN where s > m (not a candidate for that message); planes of disabled ids are left untouched.
 * The caller sizes the grid so that the surface fits.  Same stream and ownership rules as plogp_predict.
 */
int plogp_segment_surface(plogp_tables *tables, const plogp_grid *grid, double *d_surface, void *stream);

/*
 * What one fixed segment size costs (the measured Segmented Chain of the paper's Fig. 1(b) used 8 kB segments for
 * every message; Section 3.1 tunes the size instead).  For every table, segmented strategy (ids 2, 5, 9), P and m:
 *   d_time_fixed  DEVICE, double [n_tables][3][n_P][n_m]: the model with s = s_fixed, or with the whole message as
 *                 its one segment (s = m, k = 1) where s_fixed > m, as Section 3.1 sends smaller messages unsegmented
 *   d_ratio       DEVICE, double [n_tables][3][n_P][n_m]: d_time_fixed divided by the minimum over the grid's
 *                 candidates, read from d_pred_time; >= 1 wherever s_fixed is itself a candidate.  May be NULL,
 *                 together with d_pred_time.
 *   d_pred_time   DEVICE, the d_time output of plogp_predict for the same tables and the same grid
 *                 ([n_tables][13][n_P][n_m]); only the planes of the enabled segmented ids are read.
 *   s_fixed       bytes, a positive multiple of grid->dtype_bytes, < 2^32; it need not be one of the grid's candidates.
 * Planes of disabled ids are left untouched.
 */
int plogp_segment_sensitivity(plogp_tables *tables, const plogp_grid *grid, uint64_t s_fixed, const double *d_pred_time,
                              double *d_time_fixed, double *d_ratio, void *stream);

/*
 * Decision boundaries in the (P, m) plane (Sections 1 and 5: the tuner's result is a map from parameter sets to
 * strategies; this marks where the map changes).
 *   d_strategy  DEVICE, uint8 [n_tables][2][n_P][n_m], the d_strategy output of plogp_select_best
 *   d_boundary  DEVICE, uint8 [n_tables][2][n_P][n_m]: bit 0 set where the next larger process count (same m) has
 *               another strategy, bit 1 where the next larger message size (same P) has; the last row / column
 *               has no such neighbour.
 * Needs no table handle: it only reads the decision table.
 */
int plogp_decision_boundaries(int n_tables, int n_P, int n_m, const uint8_t *d_strategy, uint8_t *d_boundary, void *stream);

/* Static description of a status code. */
const char *plogp_status_string(int status);

/* Text of the CUDA error behind the calling thread's last PLOGP_E_CUDA ("" if none). */
const char *plogp_last_cuda_error(void);

/*
 * Scatter Chain predictions without any allocation.  (The paper has no counterpart for this
 * entry point: it exists for callers that must not allocate device memory while they run, such
 * as code inside a memory-pool-managed service, a real-time loop, or a section where cudaMalloc's
 * implicit device synchronisation is not acceptable.)
 *
 * Computes the Scatter Chain model, sum_{j=1..P-1} g(j m) + (P-1) L, for one pLogP table, every
 * P in P_lo..P_hi and every message size in d_m_bytes, exactly as plogp_predict does for strategy
 * id 11.  The call issues no cudaMalloc, cudaFree or other allocating routine: the partial sums of
 * its scan live in a fixed 512 KiB array inside the library image, which every device that loads
 * the library holds until the process exits.
 *   d_sizes_bytes  DEVICE, [n_bp] strictly increasing sizes (< 2^53); n_bp <= PLOGP_MAX_BREAKPOINTS
 *   d_gap          DEVICE, [n_bp] finite gaps >= 0
 *   latency        L, finite, >= 0
 *   P_lo, P_hi     process counts, 2 <= P_lo <= P_hi <= PLOGP_STATIC_MAX_P + 1 (the scan always covers the
 *                  terms j = 1 .. P_hi - 1, shared by all thread blocks, whatever P_lo is)
 *   d_m_bytes      DEVICE, [n_m] message sizes; n_m <= PLOGP_STATIC_MAX_M; P_hi * m must stay < 2^53
 *   d_time         DEVICE, [P_hi - P_lo + 1][n_m] doubles, m fastest; owned by the caller
 *   stream         cudaStream_t the three kernels are enqueued on; the call does not wait for them
 * The contents of the device arrays cannot be checked on the host and are trusted.  Sizes beyond
 * the stated maxima (n_m, P_hi - 1 <= PLOGP_STATIC_MAX_P, n_bp) return PLOGP_E_RANGE; other
 * malformed arguments PLOGP_E_INVAL.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  All calls on a device share the array, which
 * keeps the previous call's contents; each call overwrites every entry it later reads, so nothing
 * needs clearing, but two calls whose device work overlaps in time race on it: keep them on one
 * stream or order them yourself.
 */
#define PLOGP_STATIC_MAX_M 256
#define PLOGP_STATIC_MAX_P 262144
int plogp_scatter_chain_static(int n_bp, const uint64_t *d_sizes_bytes, const double *d_gap, double latency,
                               int32_t P_lo, int32_t P_hi, const uint64_t *d_m_bytes, int32_t n_m,
                               double *d_time, void *stream);

/*
 * Per-kernel device timing (measurement aid, no counterpart in the paper).  While enabled, every
 * kernel that plogp_predict / plogp_select_best launch on this handle is bracketed by two CUDA
 * events recorded on the caller's stream.  plogp_profile_read waits for the recorded events,
 * adds the elapsed milliseconds and launch counts per kernel kind into ms[PLOGP_N_KERNEL_KINDS] and
 * launches[PLOGP_N_KERNEL_KINDS] (HOST arrays), and forgets them.  Read (or free the handle)
 * regularly: each launch keeps two events alive until then.
 */
enum {
    PLOGP_KERNEL_SWEEP = 0,        /* segment sweep over long candidate lists */
    PLOGP_KERNEL_CHAIN_PREFIX = 1, /* Scatter Chain sums per tile of process counts (when P is split over thread blocks) */
    PLOGP_KERNEL_FUSED = 2,        /* all strategies, lanes <-> m (predictions, long lists' final pass) */
    PLOGP_KERNEL_DECIDE = 3,       /* Broadcast decision, lanes <-> P (short candidate lists) */
    PLOGP_KERNEL_SCATTER = 4,      /* Scatter decision */
    PLOGP_KERNEL_ENVELOPE = 5,     /* segment search by lower envelope (search_mode 1) */
    PLOGP_KERNEL_SEGMIN = 6,       /* segmented minima of plogp_predict, lanes <-> P (short candidate lists) */
    PLOGP_KERNEL_GAPS = 7,         /* g(1), g(s), g(m) once per table, in front of the lanes <-> P kernels on large grids */
    PLOGP_N_KERNEL_KINDS = 8
};
int plogp_profile_enable(plogp_tables *tables, int enable);
int plogp_profile_read(plogp_tables *tables, double *ms, int32_t *launches);

/* Number of kernels this library has launched in the calling process so far (all handles, all
 * threads).  Bookkeeping for benchmarks; no counterpart in the paper. */
uint64_t plogp_kernel_launches(void);

/*
 * Measurement aid with no counterpart in the paper: runs a register-only stream of double-precision
 * fused multiply-adds (16 independent chains per thread) on every SM of the current device for about
 * `milliseconds` and returns the sustained rate in thread-level FMA instructions per second
 * (the issue ceiling the segment sweep is compared with).  Synchronises.  Negative on error.
 */
double plogp_fp64_fma_rate(double milliseconds);

#ifdef __cplusplus
}
#endif
#endif /* PLOGP_H */
