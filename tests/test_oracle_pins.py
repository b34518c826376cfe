"""Pins of the CPU oracle against things other than itself: numpy's interpolation routine,
hand-worked values, closed forms under a linear gap, algebraic identities of Table 1 / Table 2,
and an independent lower-envelope algorithm for the segment search."""
import math
import os

import numpy as np
import pytest

from oracle import plogp_oracle as po
from paper_cs_0408034_b200 import workloads as wl

HERE = os.path.dirname(os.path.abspath(__file__))


def rand_table(seed, n_bp=9, lo=4, hi=1 << 16, L=None):
    sizes = wl.log_spaced_multiples(lo, hi, n_bp)
    gaps = wl.noisy_monotone_gaps(sizes, 3.0, 0.01, 0.3, seed)
    L = 1.0 + 20.0 * wl.uniform(seed, [999])[0] if L is None else L
    return po.Table(sizes, gaps, L)


def linear_table(a, b, sizes, L):
    sizes = np.asarray(sizes, dtype=np.uint64)
    return po.Table(sizes, a + b * sizes.astype(np.float64), L)


# ---------- g(x): Section 2, piecewise linear ----------

def test_gap_matches_numpy_interp_inside_table():
    for seed in range(5):
        t = rand_table(seed, n_bp=12)
        xs = np.unique(np.concatenate([t.sizes.astype(np.int64),
                                       (wl.uniform(seed, np.arange(400)) * float(t.sizes[-1])).astype(np.int64) + 1]))
        xs = xs[(xs >= int(t.sizes[0])) & (xs <= int(t.sizes[-1]))]
        want = np.interp(xs.astype(np.float64), t.sizes.astype(np.float64), t.gaps)
        got = np.array([po.gap(t, int(x)) for x in xs])
        np.testing.assert_allclose(got, want, rtol=1e-14, atol=0)


def test_gap_hits_breakpoints_exactly_and_clamps_below():
    t = rand_table(3)
    for s, g in zip(t.sizes, t.gaps):
        assert po.gap(t, int(s)) == g
    assert po.gap(t, 1) == t.gaps[0] and po.gap(t, 3) == t.gaps[0]


def test_gap_continues_last_line_above_table():
    t = po.Table([4, 8, 16], [2.0, 3.0, 5.0], 10.0)
    assert po.gap(t, 32) == 9.0 and po.gap(t, 48) == 13.0 and po.gap(t, 12) == 4.0


def test_gap_of_linear_table_is_the_line_everywhere():
    a, b = 7.5, 0.003
    t = linear_table(a, b, [8, 64, 1000, 4096, 65536], 1.0)
    for x in [8, 9, 63, 64, 65, 999, 5000, 65536, 65537, 10 ** 6, 10 ** 9]:
        assert po.gap(t, x) == pytest.approx(a + b * x, rel=1e-14)
    assert po.gap(t, 1) == a + b * 8


def test_log2_rounding():
    for P in range(2, 5000):
        assert po.log2_floor(P) == int(math.floor(math.log2(P) + 1e-12)) or (1 << po.log2_floor(P)) <= P < (2 << po.log2_floor(P))
        f, c = po.log2_floor(P), po.log2_ceil(P)
        assert (1 << f) <= P < (1 << (f + 1))
        assert (1 << c) >= P > (1 << (c - 1))


def test_segment_count_modes():
    assert po.segments(12, 8, 0) == 2 and po.segments(12, 8, 1) == 1
    assert po.segments(16, 8, 0) == 2 and po.segments(16, 8, 1) == 2
    assert po.segments(16, 16, 0) == 1 and po.segments(17, 16, 0) == 2


# ---------- hand-worked example (tests/golden) ----------

def test_hand_worked_example():
    t = po.Table([4, 8, 16], [2.0, 3.0, 5.0], 10.0)
    sg = po.SGrid([4, 8])
    cases = {"A": (4, 16), "B": (3, 12)}
    n = 0
    for line in open(os.path.join(HERE, "golden", "tiny_table1_table2.txt")):
        if line.startswith("#") or not line.strip():
            continue
        case, sid, k_mode, best_s, time = line.split()
        P, m = cases[case]
        sid, k_mode, best_s, time = int(sid), int(k_mode), int(best_s), float(time)
        if sid in po.SEGMENTED_IDS:
            s, v, _ = po.segment_search(t, sid, P, m, sg, k_mode)
            assert (s, v) == (best_s, time), line
        else:
            assert po.model(t, sid, P, m, 0, k_mode) == time, line
        n += 1
    assert n == 20
    # decisions of case A: flat tree wins both collectives, unsegmented
    assert po.decide(t, 0, wl.ALL_STRATEGIES, 4, 16, sg)[:3] == (0, 0, 25.0)
    assert po.decide(t, 1, wl.ALL_STRATEGIES, 4, 16, sg)[:3] == (10, 0, 25.0)
    # runner-up of the Broadcast decision is the segmented flat tree's 28
    assert po.decide(t, 0, wl.ALL_STRATEGIES, 4, 16, sg)[3] == 28.0


# ---------- identities readable off Table 1 / Table 2 ----------

def test_two_processes_collapse_to_one_transfer():
    for seed in range(4):
        t = rand_table(seed)
        for m in [4, 100, 4096, 70000]:
            one = po.gap(t, m) + t.L
            for sid in (0, 3, 7, 10, 11, 12):
                assert po.model(t, sid, 2, m) == pytest.approx(one, rel=1e-15)


def test_single_segment_equals_unsegmented():
    for seed in range(4):
        t = rand_table(seed)
        for P in [2, 3, 7, 8, 33]:
            for m in [4, 256, 5000]:
                for seg, plain in ((2, 0), (5, 3), (9, 7)):
                    assert po.model(t, seg, P, m, m) == pytest.approx(po.model(t, plain, P, m), rel=1e-15)


def test_message_below_every_candidate_goes_unsegmented():
    t = rand_table(1)
    sg = po.SGrid([1024, 2048])
    for seg, plain in ((2, 0), (5, 3), (9, 7)):
        s, v, ru = po.segment_search(t, seg, 9, 512, sg)
        assert s == 512 and ru == math.inf
        assert v == pytest.approx(po.model(t, plain, 9, 512), rel=1e-15)
    # and the unsegmented sibling (lower id) takes the tie in the decision
    sid, s, _, _ = po.decide(t, 0, (1 << 3) | (1 << 5), 9, 512, sg)
    assert (sid, s) == (3, 0)


def test_algebraic_relations_between_rows():
    t = rand_table(2)
    g1 = po.gap(t, 1)
    for P in [2, 5, 16, 100]:
        for m in [8, 1000, 60000]:
            assert po.model(t, 10, P, m) == po.model(t, 0, P, m)
            assert po.model(t, 4, P, m) - po.model(t, 3, P, m) == pytest.approx((P - 1) * (2 * g1 + 2 * t.L), rel=1e-12)
            assert po.model(t, 1, P, m) - po.model(t, 0, P, m) == pytest.approx(2 * g1 + 2 * t.L, rel=1e-12)
            lc = po.log2_ceil(P)
            assert po.model(t, 8, P, m) - po.model(t, 7, P, m) == pytest.approx(lc * (2 * g1 + 2 * t.L), rel=1e-12)
            for s in [4, 8, 64]:
                if s <= m:
                    k = -(-m // s)
                    gs = po.gap(t, s)
                    assert po.model(t, 5, P, m, s) == pytest.approx((P + k - 2) * gs + (P - 1) * t.L, rel=1e-14)
                    assert po.model(t, 2, P, m, s) == pytest.approx((P - 1) * k * gs + t.L, rel=1e-14)
                    assert po.model(t, 9, P, m, s) == pytest.approx(po.log2_floor(P) * k * gs + lc * t.L, rel=1e-14)


def test_cellwise_monotone_in_P_and_m():
    t = rand_table(4)
    ms = [4, 8, 100, 1000, 5000, 65536, 100000]
    for sid in range(13):
        for s in [4, 64]:
            prev_row = None
            for P in range(2, 40):
                row = [po.model(t, sid, P, m, s) for m in ms]
                assert all(b >= a for a, b in zip(row, row[1:])), (sid, P)
                if prev_row is not None:
                    assert all(b >= a for a, b in zip(prev_row, row)), (sid, P)
                prev_row = row


# ---------- closed forms under an exactly linear gap g(x) = a + b x ----------

A, B, LAT = 30.0, 0.08, 50.0
LIN_SIZES = [1, 16, 1024, 1 << 16, 1 << 20]


def test_scatter_chain_closed_form():
    t = linear_table(A, B, LIN_SIZES, LAT)
    for P in [2, 3, 17, 200, 3000]:
        for m in [4, 1000, 1 << 18]:
            want = (P - 1) * (A + LAT) + B * m * P * (P - 1) / 2
            assert po.model(t, 11, P, m) == pytest.approx(want, rel=1e-13)


def test_scatter_binomial_closed_form_and_crossover():
    t = linear_table(A, B, LIN_SIZES, LAT)
    sg = po.SGrid([4])
    for P in [2, 3, 8, 9, 50, 1000]:
        d = po.log2_ceil(P)
        for m in [4, 64, 1000, 1 << 16]:
            want = d * A + B * m * (2 ** d - 1) + d * LAT
            assert po.model(t, 12, P, m) == pytest.approx(want, rel=1e-13)
            lhs, rhs = (P - 1 - d) * A, (d - 1) * LAT + B * m * (2 ** d - P)
            if abs(lhs - rhs) > 1e-6 * max(lhs, rhs, 1.0):
                sid = po.decide(t, 1, (1 << 10) | (1 << 12), P, m, sg)[0]
                assert sid == (12 if lhs > rhs else 10), (P, m)


def test_pipelined_chain_optimal_segment_brackets_closed_form():
    t = linear_table(A, B, LIN_SIZES, LAT)
    s_grid = [1 << e for e in range(2, 21)]
    sg = po.SGrid(s_grid)
    for P in [3, 4, 10, 50, 500]:
        for m in [1 << 12, 1 << 16, 1 << 20]:
            s_star = math.sqrt(A * m / ((P - 2) * B))
            s, _, _ = po.segment_search(t, 5, P, m, sg)
            cands = [x for x in s_grid if x <= m]
            below = max([x for x in cands if x <= s_star], default=cands[0])
            above = min([x for x in cands if x >= s_star], default=cands[-1])
            assert s in (below, above), (P, m, s, s_star)
    # two processes: no pipeline to fill, the whole message in one segment wins
    for m in [1 << 12, 1 << 20]:
        assert po.segment_search(t, 5, 2, m, sg)[0] == m


def test_qualitative_outcome_on_ethernet_like_network():
    """Section 4.1: on the 100 Mbit/s network the Segmented Chain beats the Binomial Broadcast."""
    t = linear_table(30.0, 0.08, [1 << e for e in range(21)], 50.0)
    seg = po.model(t, 5, 50, 1 << 20, 8192)
    bino = po.model(t, 7, 50, 1 << 20)
    assert seg == pytest.approx(49 * (685.36 + 50) + 685.36 * 127, rel=1e-12)
    assert bino == pytest.approx(5 * (30 + 0.08 * 2 ** 20) + 6 * 50, rel=1e-12)
    assert seg < bino / 3


# ---------- independent algorithm for the segment search: lower envelope of lines in P ----------

def _envelope_argmin(lines, P_values):
    """lines: (A, B, s) meaning T(P) = A + B*P. Brute force is avoided: sort by slope, build the
    lower hull, then walk it with P ascending. Returns the (time, s) per P."""
    lines = sorted(lines, key=lambda l: (-l[1], l[0], l[2]))  # steepest first: optimal for small P
    hull = []

    def bad(l1, l2, l3):
        # l2 is never strictly below both neighbours
        return (l3[0] - l1[0]) * (l1[1] - l2[1]) <= (l2[0] - l1[0]) * (l1[1] - l3[1])

    for l in lines:
        if hull and hull[-1][1] == l[1]:
            continue  # same slope, higher (or equal) intercept
        while len(hull) >= 2 and bad(hull[-2], hull[-1], l):
            hull.pop()
        hull.append(l)
    out, i = [], 0
    for P in P_values:
        while i + 1 < len(hull) and hull[i + 1][0] + hull[i + 1][1] * P <= hull[i][0] + hull[i][1] * P:
            i += 1
        out.append((hull[i][0] + hull[i][1] * P, hull[i][2]))
    return out


def test_segment_search_against_lower_envelope():
    w = wl.config3(P_hi=300, n_m=6, m_lo=4 << 10, m_hi=1 << 16, s_hi=1 << 14)
    t = po.Table(w.sizes, w.gaps[0], w.latency[0])
    sg = po.SGrid(lo=w.s_lo, hi=w.s_hi, step=w.s_step)
    Ps = list(range(2, 301))
    checked = 0
    for m in [int(x) for x in w.m]:
        lines = []
        for s in range(4, min(m, w.s_hi) + 1, 4):
            gs = po.gap(t, s)
            k = -(-m // s)
            lines.append(((k - 2) * gs - t.L, gs + t.L, s))
        env = _envelope_argmin(lines, Ps)
        for P, (tv, s_env) in zip(Ps, env):
            s, v, ru = po.segment_search(t, 5, P, m, sg)
            assert v == pytest.approx(tv, rel=1e-12)
            if (ru - v) / v > 1e-9:
                assert s == s_env, (P, m)
                checked += 1
    assert checked > 200


# ---------- the grid evaluators agree with the one-cell functions ----------

def test_grid_equals_cellwise():
    w = wl.config1()
    t = po.Table(w.sizes, w.gaps[0], w.latency[0])
    sg = po.SGrid(w.s_list)
    mask = wl.ALL_STRATEGIES
    pred = po.predict_grid(t, mask, w.P_values(), w.m, sg)
    dec = po.select_grid(mask, pred)
    for ip in (0, 1, 7, 30, 48):
        for im in (0, 5, 9, 12, 18):
            P, m = int(w.P_values()[ip]), int(w.m[im])
            for sid in range(13):
                if sid in po.SEGMENTED_IDS:
                    s, v, ru = po.segment_search(t, sid, P, m, sg)
                    q = po.SEGMENTED_IDS.index(sid)
                    assert pred.best_s[q, ip, im] == s and pred.seg_runner_up[q, ip, im] == ru
                else:
                    v = po.model(t, sid, P, m)
                assert pred.time[sid, ip, im] == v, (sid, P, m)
            for c in (0, 1):
                sid, s, v, ru = po.decide(t, c, mask, P, m, sg)
                assert (dec.strategy[c, ip, im], dec.s[c, ip, im], dec.time[c, ip, im], dec.runner_up[c, ip, im]) == (sid, s, v, ru)
