/*
 * plogp_oracle.h — CPU oracle for the pLogP collective-communication cost models.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, host-only evaluator of the
 * models printed in Table 1 (Broadcast) and Table 2 (Scatter) of "Fast Tuning of
 * Intra-Cluster Collective Communications" (Barchet-Estefanel & Mounié), followed
 * by the exhaustive segment-size search of Section 3.1 and the per-parameter-set
 * strategy selection of Sections 1 and 5.  It shares no code with the CUDA
 * library and must never be linked, imported or executed by the product path;
 * only the test-suite, the smoke check and the CPU-baseline leg of the benchmark
 * may use it.
 *
 * Everything is evaluated in IEEE double, one cell at a time, in the order the
 * tables print the terms; the Scatter sums are accumulated in `long double` and
 * rounded to double once.
 *
 * Readings taken where the paper is silent (both this oracle and the CUDA path
 * follow them; the paper does not pin them — "parity unpinned" for these):
 *   - g(x) between measured sizes: linear in x (bytes) between neighbouring
 *     breakpoints; below the first breakpoint g is held at its first value;
 *     above the last breakpoint the last interval's line is continued.
 *   - k, the number of segments (Section 2: s splits m into k segments):
 *     k = ceil(m/s) by default (k_mode 0), floor(m/s) as Section 3.1 prints it
 *     (k_mode 1).  Every segment is charged g(s), as Table 1 prints g(s) x k.
 *   - candidate segment sizes for a message m are the grid values s <= m; when
 *     there is none the message goes unsegmented (Section 3.1), evaluated as
 *     s = m, k = 1.
 *   - ties: smallest segment size, then lowest strategy id (Table order).
 *
 * Strategy ids (Table 1 rows, then Table 2 rows):
 *   0 Flat Tree                 5 Segmented Chain (Pipeline)   10 Scatter Flat Tree
 *   1 Flat Tree Rendezvous      6 Binary Tree                  11 Scatter Chain
 *   2 Segmented Flat Tree       7 Binomial Tree                12 Scatter Binomial Tree
 *   3 Chain                     8 Binomial Tree Rendezvous
 *   4 Chain Rendezvous          9 Segmented Binomial Tree
 *
 * Collectives the paper names but prints no models for (Section 3: Barrier, Reduce and Gather are built "in a very
 * similar way" as Broadcast and Scatter).  Their models here are derived, not printed: with the gap charged to a
 * node's port for receives as for sends (in Table 1 / Table 2 no node ever receives two messages at once, so the
 * paper never needs that rule), a Gather is a Scatter run backwards in time and a Reduce a Broadcast run backwards
 * (communication only: pLogP has no parameter for the combine operation), so their times are those of the mirrored
 * strategy; a Barrier is a Reduce followed by a Broadcast of one-byte messages, g(1) being the gap the paper's
 * rendezvous rows already use for an empty message.  "parity unpinned" by the paper; pinned here by the
 * send-schedule simulation with a receive port.
 *  13 Gather Flat Tree          (P-1) g(m) + L                                   (= id 10)
 *  14 Gather Chain              sum_{j=1..P-1} g(j m) + (P-1) L                  (= id 11)
 *  15 Gather Binomial Tree      sum_{j=0..ceil(log2 P)-1} g(2^j m) + ceil(log2 P) L   (= id 12)
 *  16 Reduce Flat Tree (= 0)    17 Reduce Segmented Flat Tree (= 2)   18 Reduce Chain (= 3)
 *  19 Reduce Segmented Chain (= 5)   20 Reduce Binary Tree (= 6)   21 Reduce Binomial Tree (= 7)
 *  22 Reduce Segmented Binomial Tree (= 9)
 *  23 Barrier Flat Tree         2 ((P-1) g(1) + L)
 *  24 Barrier Chain             2 (P-1) (g(1) + L)
 *  25 Barrier Binary Tree       2 ceil(log2 P) (2 g(1) + L)
 *  26 Barrier Binomial Tree     2 (floor(log2 P) g(1) + ceil(log2 P) L)
 */
#ifndef PLOGP_ORACLE_H
#define PLOGP_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PO_N_STRATEGIES 13
#define PO_N_SEGMENTED 3 /* ids 2, 5, 9 in this order */

/* One measured pLogP parameter set (Section 2): gap g at n_bp message sizes, latency L. */
typedef struct {
    int n_bp;
    const uint64_t *size; /* [n_bp] bytes, strictly increasing */
    const double *gap;    /* [n_bp] */
    double L;
} po_table;

/* Candidate segment sizes: an explicit ascending list (list != NULL) or every
 * lo + i*step <= hi. */
typedef struct {
    const uint64_t *list;
    int64_t n_list;
    uint64_t lo, hi, step;
} po_sgrid;

/* g(x): Section 2 "gap of a message of size x", evaluated on the table. */
double po_gap(const po_table *t, uint64_t x);

int po_log2_floor(int64_t P);
int po_log2_ceil(int64_t P);

/* k of Section 2 / Section 3.1 for message m and segment s (s <= m or s == m). */
uint64_t po_segments(uint64_t m, uint64_t s, int k_mode);

/* One model cell exactly as Table 1 / Table 2 print it.  s is ignored by the
 * unsegmented strategies.  Returns NaN for an unknown id. */
double po_model(const po_table *t, int strategy, int64_t P, uint64_t m, uint64_t s, int k_mode);

/* Section 3.1 search: over the candidates s <= m (or s = m when none) return
 * the smallest s attaining the minimum of the model, that minimum, and the
 * smallest time among the OTHER candidates (+inf when there is only one). */
void po_segment_search(const po_table *t, int strategy, int64_t P, uint64_t m, const po_sgrid *sg,
                       int k_mode, uint64_t *best_s, double *best_time, double *runner_up);

/* Strategy selection for one (collective, P, m): collective 0 = Broadcast
 * (ids 0..9), 1 = Scatter (ids 10..12), 2 = Gather (13..15), 3 = Reduce (16..22), 4 = Barrier (23..26, m is
 * ignored); only ids enabled in mask (bit i = id i) compete.
 * s_out = 0 when the winner is unsegmented.  runner_up = best time of the
 * best OTHER strategy (+inf if none).  Returns 0, or -1 when no strategy of
 * that collective is enabled (outputs untouched). */
int po_decide(const po_table *t, int collective, uint32_t mask, int64_t P, uint64_t m,
              const po_sgrid *sg, int k_mode, int *strategy_out, uint64_t *s_out, double *time_out,
              double *runner_up);

/* Whole grids (OpenMP over cells).  Layouts, with m fastest:
 *   time     [13][n_P][n_m]   (disabled strategies left untouched)
 *   best_s   [3][n_P][n_m]    (ids 2, 5, 9)
 *   seg_ru   [3][n_P][n_m]    runner-up time over the other segment sizes
 * The Scatter Chain column is accumulated incrementally along ascending P
 * (the same long-double sum, not restarted for every P). */
void po_predict_grid(const po_table *t, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m,
                     int n_m, const po_sgrid *sg, int k_mode, double *time, uint64_t *best_s,
                     double *seg_ru);

/* Decision table from a predicted grid: for collective c in {0,1}
 *   strategy [2][n_P][n_m] (255 when nothing enabled), s [2][..], time [2][..],
 *   runner_up [2][..] (best time of the best other strategy). */
void po_select_grid(uint32_t mask, int n_P, int n_m, const double *time, const uint64_t *best_s,
                    uint8_t *strategy, uint64_t *s_out, double *time_out, double *runner_up);

/* ---- Sensitivity to the segment size (Section 3.1; the measured Segmented Chain of Fig. 1(b) used 8 kB) ----
 *
 * The segment size a fixed setting really uses for a message m: s_fixed itself when it fits (s_fixed <= m),
 * otherwise the whole message (s = m, one segment), as Section 3.1 sends smaller messages unsegmented. */
uint64_t po_effective_segment(uint64_t m, uint64_t s_fixed);

/* Model surface over s: out[q][ip][im][is] = po_model(id_q, P[ip], m[im], s_is) for the segmented ids
 * q = 0,1,2 (2, 5, 9) enabled in mask and every candidate s_is of the grid; NaN where s_is > m[im]
 * (not a candidate for that message) or the id is disabled.  n_s = number of candidates of sg. */
void po_surface_grid(const po_table *t, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m, int n_m,
                     const po_sgrid *sg, int k_mode, double *out);

/* time_fixed[q][ip][im] = po_model(id_q, P, m, po_effective_segment(m, s_fixed)); disabled ids untouched. */
void po_fixed_segment_grid(const po_table *t, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m,
                           int n_m, uint64_t s_fixed, int k_mode, double *time_fixed);

/* po_decide over a grid (OpenMP over cells): strategy / s / time / runner_up, each [n_P][n_m]. */
void po_decide_grid(const po_table *t, int collective, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m, int n_m,
                    const po_sgrid *sg, int k_mode, uint8_t *strategy, uint64_t *s_out, double *time_out, double *runner_up);

#define PO_N_MODELS 27

int po_threads(void);

#ifdef __cplusplus
}
#endif
#endif
