"""Pins of the oracle's segment-size sensitivity functions (model surface over s, fixed segment size, decision
boundaries) against things other than themselves: discrete-event simulation of the send schedules, the
closed forms under a linear gap, the one-segment identity, the exhaustive search of Section 3.1 and a
hand-made boundary map."""
import numpy as np
import pytest

import des
from oracle import plogp_oracle as po
from paper_cs_0408034_b200 import workloads as wl

SEG = (2, 5, 9)
MASK = sum(1 << i for i in SEG)


def small_table(seed=3):
    sizes = wl.log_spaced_multiples(4, 1 << 16, 12)
    gaps = wl.noisy_monotone_gaps(sizes, 3.0, 0.01, 0.05, seed)
    return po.Table(sizes, gaps, 7.0)


def test_surface_cells_equal_the_simulated_send_schedules():
    """Segmented Flat Tree and Segmented Chain at every P, Segmented Binomial at powers of two: each surface cell is
    the completion time of the strategy's pLogP send schedule with k segments of size s."""
    t = small_table()
    sg = po.SGrid([4, 16, 64, 256])
    P = [2, 3, 4, 7, 8]
    m = [64, 256, 1024]
    surf = po.surface_grid(t, MASK, P, m, sg)
    g = lambda x: po.gap(t, x)
    for ip, Pv in enumerate(P):
        for im, mv in enumerate(m):
            for js, s in enumerate([4, 16, 64, 256]):
                if s > mv:
                    assert np.isnan(surf[:, ip, im, js]).all()
                    continue
                k = po.segments(mv, s)
                assert surf[0, ip, im, js] == pytest.approx(des.simulate(Pv, des.segmented_flat(Pv, s, k), g, t.L), rel=1e-12)
                assert surf[1, ip, im, js] == pytest.approx(des.simulate(Pv, des.segmented_chain(Pv, s, k), g, t.L), rel=1e-12)
                if Pv & (Pv - 1) == 0:
                    assert surf[2, ip, im, js] == pytest.approx(des.simulate(Pv, des.segmented_binomial(Pv, s, k), g, t.L), rel=1e-12)


def test_surface_closed_forms_under_a_linear_gap():
    a, b, L = 4.0, 0.002, 9.0
    sizes = np.array([4, 1 << 10, 1 << 22], dtype=np.uint64)
    t = po.Table(sizes, a + b * sizes.astype(np.float64), L)
    s = np.array([64, 256, 4096, 65536], dtype=np.uint64)
    P = np.array([2, 5, 16, 33])
    m = np.array([65536, 1 << 20], dtype=np.uint64)   # every s divides every m
    surf = po.surface_grid(t, MASK, P, m, po.SGrid(s))
    Pm1 = (P - 1.0)[:, None, None]
    lf = np.floor(np.log2(P))[:, None, None]
    lc = np.ceil(np.log2(P))[:, None, None]
    gs = (a + b * s.astype(np.float64))[None, None, :]
    k = m.astype(np.float64)[None, :, None] / s.astype(np.float64)[None, None, :]
    np.testing.assert_allclose(surf[0], Pm1 * gs * k + L, rtol=1e-12)
    np.testing.assert_allclose(surf[1], Pm1 * (gs + L) + gs * (k - 1.0), rtol=1e-12)
    np.testing.assert_allclose(surf[2], lf * gs * k + lc * L, rtol=1e-12)


def test_minimum_of_the_surface_is_the_exhaustive_search():
    t = small_table(5)
    s = wl.log_spaced_multiples(4, 1 << 14, 17)
    sg = po.SGrid(s)
    P = [2, 9, 40, 300]
    m = [4, 100, 5000, 1 << 15]
    for k_mode in (0, 1):
        surf = po.surface_grid(t, MASK, P, m, sg, k_mode)
        for q, sid in enumerate(SEG):
            for ip, Pv in enumerate(P):
                for im, mv in enumerate(m):
                    bs, bt, _ = po.segment_search(t, sid, Pv, mv, sg, k_mode)
                    row = surf[q, ip, im]
                    if np.isnan(row).all():      # no candidate fits: the search sends the message whole
                        assert bs == mv
                        continue
                    j = int(np.nanargmin(row))    # first minimum = smallest s
                    assert row[j] == bt and int(s[j]) == bs
                    assert np.isnan(row[s > mv]).all() and not np.isnan(row[s <= mv]).any()


def test_fixed_segment_size_one_segment_identity_and_ratio():
    t = small_table(9)
    P = [2, 3, 17, 64]
    m = [4, 512, 8192, 1 << 16]
    sg = po.SGrid(wl.log_spaced_multiples(4, 1 << 14, 15))
    # a fixed size that no message reaches: every message goes whole, i.e. the unsegmented sibling's time
    whole = po.fixed_segment_grid(t, MASK, P, m, 1 << 20)
    for q, sibling in enumerate((0, 3, 7)):
        for ip, Pv in enumerate(P):
            for im, mv in enumerate(m):
                assert whole[q, ip, im] == po.model(t, sibling, Pv, mv)
    assert po.effective_segment(100, 64) == 64 and po.effective_segment(100, 128) == 100 and po.effective_segment(64, 64) == 64
    # a fixed size taken from the candidate list can never beat the search, and equals it where it is the optimum
    s_fixed = int(sg.values[9])
    fixed = po.fixed_segment_grid(t, MASK, P, m, s_fixed)
    pred = po.predict_grid(t, MASK, P, m, sg)
    for q, sid in enumerate(SEG):
        ratio = fixed[q] / pred.time[sid]
        fits = np.array(m)[None, :] >= s_fixed
        assert (ratio[np.broadcast_to(fits, ratio.shape)] >= 1.0).all()
        hit = pred.best_s[q] == s_fixed
        assert (ratio[hit] == 1.0).all()
    # disabled strategies are left alone
    only5 = po.fixed_segment_grid(t, 1 << 5, P, m, s_fixed)
    assert np.isnan(only5[0]).all() and np.isnan(only5[2]).all() and not np.isnan(only5[1]).any()


def test_decision_boundaries_on_a_hand_made_map():
    s = np.array([[1, 1, 2],
                  [1, 3, 3]])
    assert po.decision_boundaries(s).tolist() == [[0, 3, 1], [2, 0, 0]]
    rng = np.random.default_rng(1)
    big = rng.integers(0, 3, size=(2, 9, 11))
    b = po.decision_boundaries(big)
    for c in range(2):
        for ip in range(9):
            changes = sum(big[c, ip, j] != big[c, ip, j + 1] for j in range(10))
            assert int(((b[c, ip] >> 1) & 1).sum()) == changes
        for im in range(11):
            changes = sum(big[c, j, im] != big[c, j + 1, im] for j in range(8))
            assert int((b[c, :, im] & 1).sum()) == changes
