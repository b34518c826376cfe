/*
 * plogp_oracle.c — see plogp_oracle.h.  TEST INFRASTRUCTURE ONLY: a plain CPU
 * evaluator of the paper's Table 1 / Table 2 models, the Section 3.1 segment
 * search and the strategy selection.  No blocking, no hoisting beyond what the
 * definitions state; one cell at a time.
 */
#include "plogp_oracle.h"

#include <math.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- Section 2: g(x) on a measured table (piecewise linear in bytes) ---- */
double po_gap(const po_table *t, uint64_t x)
{
    const int n = t->n_bp;
    if (x <= t->size[0]) return t->gap[0]; /* held at the first measured value below the table */
    /* interval i with size[i] <= x, the last interval also serving x beyond the table */
    int i = n - 2;
    while (i > 0 && t->size[i] > x) --i;
    double dx = (double)(x - t->size[i]);
    double dg = t->gap[i + 1] - t->gap[i];
    double dm = (double)(t->size[i + 1] - t->size[i]);
    return t->gap[i] + dx * dg / dm;
}

int po_log2_floor(int64_t P)
{
    int e = 0;
    while ((P >> (e + 1)) != 0) ++e;
    return e;
}

int po_log2_ceil(int64_t P)
{
    int e = 0;
    while (((int64_t)1 << e) < P) ++e;
    return e;
}

/* ---- Section 2 / 3.1: number of segments ---- */
uint64_t po_segments(uint64_t m, uint64_t s, int k_mode)
{
    uint64_t k = m / s;
    if (k_mode == 0 && k * s != m) ++k;
    return k;
}

/* ---- Table 1 and Table 2, one cell, as printed ---- */
double po_model(const po_table *t, int strategy, int64_t P, uint64_t m, uint64_t s, int k_mode)
{
    const double L = t->L;
    const double Pm1 = (double)(P - 1);
    const double lf = (double)po_log2_floor(P);
    const double lc = (double)po_log2_ceil(P);
    switch (strategy) {
    case 0: /* Flat Tree: (P-1) g(m) + L */
        return Pm1 * po_gap(t, m) + L;
    case 1: /* Flat Tree Rendezvous: (P-1) g(m) + 2 g(1) + 3 L */
        return Pm1 * po_gap(t, m) + 2.0 * po_gap(t, 1) + 3.0 * L;
    case 2: { /* Segmented Flat Tree: (P-1) (g(s) k) + L */
        double k = (double)po_segments(m, s, k_mode);
        return Pm1 * (po_gap(t, s) * k) + L;
    }
    case 3: /* Chain: (P-1) (g(m) + L) */
        return Pm1 * (po_gap(t, m) + L);
    case 4: /* Chain Rendezvous: (P-1) (g(m) + 2 g(1) + 3 L) */
        return Pm1 * (po_gap(t, m) + 2.0 * po_gap(t, 1) + 3.0 * L);
    case 5: { /* Segmented Chain: (P-1) (g(s) + L) + g(s) (k-1) */
        double k = (double)po_segments(m, s, k_mode);
        double gs = po_gap(t, s);
        return Pm1 * (gs + L) + gs * (k - 1.0);
    }
    case 6: /* Binary Tree: the printed upper bound, ceil(log2 P) (2 g(m) + L), taken as the prediction */
        return lc * (2.0 * po_gap(t, m) + L);
    case 7: /* Binomial Tree: floor(log2 P) g(m) + ceil(log2 P) L */
        return lf * po_gap(t, m) + lc * L;
    case 8: /* Binomial Tree Rendezvous: floor(log2 P) g(m) + ceil(log2 P) (2 g(1) + 3 L) */
        return lf * po_gap(t, m) + lc * (2.0 * po_gap(t, 1) + 3.0 * L);
    case 9: { /* Segmented Binomial Tree: floor(log2 P) g(s) k + ceil(log2 P) L */
        double k = (double)po_segments(m, s, k_mode);
        return lf * po_gap(t, s) * k + lc * L;
    }
    case 10: /* Scatter Flat Tree: (P-1) g(m) + L */
        return Pm1 * po_gap(t, m) + L;
    case 11: { /* Scatter Chain: sum_{j=1}^{P-1} g(j m) + (P-1) L */
        long double acc = 0.0L;
        for (int64_t j = 1; j <= P - 1; ++j) acc += (long double)po_gap(t, (uint64_t)j * m);
        return (double)acc + Pm1 * L;
    }
    case 12: { /* Scatter Binomial Tree: sum_{j=0}^{ceil(log2 P)-1} g(2^j m) + ceil(log2 P) L */
        long double acc = 0.0L;
        int d = po_log2_ceil(P);
        for (int j = 0; j < d; ++j) acc += (long double)po_gap(t, ((uint64_t)1 << j) * m);
        return (double)acc + lc * L;
    }
    /* ---- derived collectives (see the header): mirrored strategies, and a Barrier of one-byte messages ---- */
    case 13: return po_model(t, 10, P, m, s, k_mode); /* Gather Flat Tree */
    case 14: return po_model(t, 11, P, m, s, k_mode); /* Gather Chain */
    case 15: return po_model(t, 12, P, m, s, k_mode); /* Gather Binomial Tree */
    case 16: return po_model(t, 0, P, m, s, k_mode);  /* Reduce Flat Tree */
    case 17: return po_model(t, 2, P, m, s, k_mode);  /* Reduce Segmented Flat Tree */
    case 18: return po_model(t, 3, P, m, s, k_mode);  /* Reduce Chain */
    case 19: return po_model(t, 5, P, m, s, k_mode);  /* Reduce Segmented Chain */
    case 20: return po_model(t, 6, P, m, s, k_mode);  /* Reduce Binary Tree */
    case 21: return po_model(t, 7, P, m, s, k_mode);  /* Reduce Binomial Tree */
    case 22: return po_model(t, 9, P, m, s, k_mode);  /* Reduce Segmented Binomial Tree */
    case 23: /* Barrier Flat Tree: 2 ((P-1) g(1) + L) */
        return 2.0 * (Pm1 * po_gap(t, 1) + L);
    case 24: /* Barrier Chain: 2 (P-1) (g(1) + L) */
        return 2.0 * (Pm1 * (po_gap(t, 1) + L));
    case 25: /* Barrier Binary Tree: 2 ceil(log2 P) (2 g(1) + L) */
        return 2.0 * (lc * (2.0 * po_gap(t, 1) + L));
    case 26: /* Barrier Binomial Tree: 2 (floor(log2 P) g(1) + ceil(log2 P) L) */
        return 2.0 * (lf * po_gap(t, 1) + lc * L);
    default:
        return NAN;
    }
}

/* ---- Section 3.1: exhaustive search of the segment size ---- */
static int64_t sgrid_count(const po_sgrid *sg)
{
    if (sg->list) return sg->n_list;
    if (sg->step == 0 || sg->hi < sg->lo) return 0;
    return (int64_t)((sg->hi - sg->lo) / sg->step) + 1;
}

static uint64_t sgrid_at(const po_sgrid *sg, int64_t i)
{
    return sg->list ? sg->list[i] : sg->lo + (uint64_t)i * sg->step;
}

void po_segment_search(const po_table *t, int strategy, int64_t P, uint64_t m, const po_sgrid *sg,
                       int k_mode, uint64_t *best_s, double *best_time, double *runner_up)
{
    double bt = INFINITY, ru = INFINITY;
    uint64_t bs = 0;
    int64_t n = sgrid_count(sg);
    int any = 0;
    for (int64_t i = 0; i < n; ++i) {
        uint64_t s = sgrid_at(sg, i);
        if (s > m) break; /* ascending: nothing further fits in the message */
        double v = po_model(t, strategy, P, m, s, k_mode);
        any = 1;
        if (v < bt) {
            ru = bt;
            bt = v;
            bs = s;
        } else if (v < ru) {
            ru = v;
        }
    }
    if (!any) { /* message smaller than every candidate: sent whole */
        bs = m;
        bt = po_model(t, strategy, P, m, m, k_mode);
        ru = INFINITY;
    }
    *best_s = bs;
    *best_time = bt;
    *runner_up = ru;
}

static int is_segmented(int id) { return id == 2 || id == 5 || id == 9 || id == 17 || id == 19 || id == 22; }

/* ---- Sections 1 and 5: pick the strategy with the lowest prediction ---- */
int po_decide(const po_table *t, int collective, uint32_t mask, int64_t P, uint64_t m,
              const po_sgrid *sg, int k_mode, int *strategy_out, uint64_t *s_out, double *time_out,
              double *runner_up)
{
    static const int first[6] = {0, 10, 13, 16, 23, 27};
    if (collective < 0 || collective > 4) return -1;
    int lo = first[collective], hi = first[collective + 1];
    double bt = INFINITY, ru = INFINITY;
    int bid = -1;
    uint64_t bs = 0;
    for (int id = lo; id < hi; ++id) {
        if (!((mask >> id) & 1u)) continue;
        double v, dummy;
        uint64_t s = 0;
        if (is_segmented(id))
            po_segment_search(t, id, P, m, sg, k_mode, &s, &v, &dummy);
        else
            v = po_model(t, id, P, m, 0, k_mode);
        if (v < bt) {
            ru = bt;
            bt = v;
            bid = id;
            bs = s;
        } else if (v < ru) {
            ru = v;
        }
    }
    if (bid < 0) return -1;
    *strategy_out = bid;
    *s_out = bs;
    *time_out = bt;
    *runner_up = ru;
    return 0;
}

/* ---- whole grids ---- */
void po_predict_grid(const po_table *t, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m,
                     int n_m, const po_sgrid *sg, int k_mode, double *time, uint64_t *best_s,
                     double *seg_ru)
{
    const size_t plane = (size_t)n_P * (size_t)n_m;
    static const int seg_ids[PO_N_SEGMENTED] = {2, 5, 9};

#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int ip = 0; ip < n_P; ++ip) {
        for (int im = 0; im < n_m; ++im) {
            size_t cell = (size_t)ip * n_m + im;
            for (int id = 0; id < PO_N_STRATEGIES; ++id) {
                if (!((mask >> id) & 1u) || is_segmented(id) || id == 11) continue;
                time[id * plane + cell] = po_model(t, id, P[ip], m[im], 0, k_mode);
            }
            for (int q = 0; q < PO_N_SEGMENTED; ++q) {
                int id = seg_ids[q];
                if (!((mask >> id) & 1u)) continue;
                uint64_t s;
                double v, ru;
                po_segment_search(t, id, P[ip], m[im], sg, k_mode, &s, &v, &ru);
                time[id * plane + cell] = v;
                if (best_s) best_s[q * plane + cell] = s;
                if (seg_ru) seg_ru[q * plane + cell] = ru;
            }
        }
    }

    /* Scatter Chain: the sum over j = 1..P-1 grows with P; keep one running
     * long-double sum per message size and read it off at every listed P. */
    if ((mask >> 11) & 1u) {
#pragma omp parallel for schedule(dynamic, 1)
        for (int im = 0; im < n_m; ++im) {
            long double acc = 0.0L;
            int64_t j = 1;
            for (int ip = 0; ip < n_P; ++ip) {
                for (; j <= P[ip] - 1; ++j) acc += (long double)po_gap(t, (uint64_t)j * m[im]);
                time[11 * plane + (size_t)ip * n_m + im] = (double)acc + (double)(P[ip] - 1) * t->L;
            }
        }
    }
}

void po_select_grid(uint32_t mask, int n_P, int n_m, const double *time, const uint64_t *best_s,
                    uint8_t *strategy, uint64_t *s_out, double *time_out, double *runner_up)
{
    const size_t plane = (size_t)n_P * (size_t)n_m;
#pragma omp parallel for schedule(static)
    for (int64_t cell = 0; cell < (int64_t)plane; ++cell) {
        for (int c = 0; c < 2; ++c) {
            int lo = c == 0 ? 0 : 10, hi = c == 0 ? 10 : 13;
            double bt = INFINITY, ru = INFINITY;
            int bid = 255;
            uint64_t bs = 0;
            for (int id = lo; id < hi; ++id) {
                if (!((mask >> id) & 1u)) continue;
                double v = time[id * plane + cell];
                if (v < bt) {
                    ru = bt;
                    bt = v;
                    bid = id;
                    bs = id == 2 ? best_s[0 * plane + cell]
                         : id == 5 ? best_s[1 * plane + cell]
                         : id == 9 ? best_s[2 * plane + cell]
                                   : 0;
                } else if (v < ru) {
                    ru = v;
                }
            }
            strategy[c * plane + cell] = (uint8_t)bid;
            s_out[c * plane + cell] = bs;
            time_out[c * plane + cell] = bt;
            runner_up[c * plane + cell] = ru;
        }
    }
}

/* ---- Sensitivity to the segment size ---- */
uint64_t po_effective_segment(uint64_t m, uint64_t s_fixed) { return s_fixed <= m ? s_fixed : m; }

void po_surface_grid(const po_table *t, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m, int n_m,
                     const po_sgrid *sg, int k_mode, double *out)
{
    static const int seg_ids[PO_N_SEGMENTED] = {2, 5, 9};
    const int64_t n_s = sgrid_count(sg);
    for (int q = 0; q < PO_N_SEGMENTED; ++q)
        for (int ip = 0; ip < n_P; ++ip)
            for (int im = 0; im < n_m; ++im)
                for (int64_t is = 0; is < n_s; ++is) {
                    uint64_t s = sgrid_at(sg, is);
                    double v = NAN;
                    if (((mask >> seg_ids[q]) & 1u) && s <= m[im]) v = po_model(t, seg_ids[q], P[ip], m[im], s, k_mode);
                    out[(((size_t)q * n_P + ip) * n_m + im) * (size_t)n_s + (size_t)is] = v;
                }
}

void po_fixed_segment_grid(const po_table *t, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m,
                           int n_m, uint64_t s_fixed, int k_mode, double *time_fixed)
{
    static const int seg_ids[PO_N_SEGMENTED] = {2, 5, 9};
    for (int q = 0; q < PO_N_SEGMENTED; ++q) {
        if (!((mask >> seg_ids[q]) & 1u)) continue;
        for (int ip = 0; ip < n_P; ++ip)
            for (int im = 0; im < n_m; ++im)
                time_fixed[((size_t)q * n_P + ip) * n_m + im] =
                    po_model(t, seg_ids[q], P[ip], m[im], po_effective_segment(m[im], s_fixed), k_mode);
    }
}

void po_decide_grid(const po_table *t, int collective, uint32_t mask, const int64_t *P, int n_P, const uint64_t *m, int n_m,
                    const po_sgrid *sg, int k_mode, uint8_t *strategy, uint64_t *s_out, double *time_out, double *runner_up)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int ip = 0; ip < n_P; ++ip)
        for (int im = 0; im < n_m; ++im) {
            size_t cell = (size_t)ip * n_m + im;
            int id = 255;
            uint64_t s = 0;
            double v = NAN, ru = NAN;
            if (po_decide(t, collective, mask, P[ip], m[im], sg, k_mode, &id, &s, &v, &ru) != 0) id = 255;
            strategy[cell] = (uint8_t)id;
            s_out[cell] = s;
            time_out[cell] = v;
            runner_up[cell] = ru;
        }
}

int po_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
