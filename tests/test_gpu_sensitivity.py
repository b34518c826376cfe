"""plogp_segment_surface, plogp_segment_sensitivity and plogp_decision_boundaries through the C ABI against the
CPU oracle: times within 1e-12 relative, NaN patterns and boundary flags bit for bit."""
import numpy as np
import pytest

from paper_cs_0408034_b200 import workloads as wl
from parity import oracle_sgrid, oracle_tables

pytestmark = pytest.mark.gpu
RTOL = 1e-12


@pytest.fixture(scope="module")
def plogp():
    import torch
    assert torch.cuda.is_available()
    from paper_cs_0408034_b200 import plogp as mod
    return mod


def check_surface(plogp, w, tables=None):
    import torch
    from oracle import plogp_oracle as po
    ot = oracle_tables(w)
    with plogp.Tables.from_workload(w) as tabs:
        surf = plogp.segment_surface(tabs, w)
        torch.cuda.synchronize()
    got = surf.cpu().numpy()
    for t in (range(w.n_tables) if tables is None else tables):
        want = po.surface_grid(ot[t], w.strategy_mask, w.P_values(), w.m, oracle_sgrid(w), w.k_mode)
        for q, sid in enumerate((2, 5, 9)):
            if not (w.strategy_mask >> sid) & 1:
                assert np.isinf(got[t, q]).all()          # untouched (the binding pre-fills with inf)
                continue
            nan_w, nan_g = np.isnan(want[q]), np.isnan(got[t, q])
            assert np.array_equal(nan_w, nan_g)
            ok = ~nan_w
            assert (np.abs(got[t, q][ok] - want[q][ok]) <= RTOL * want[q][ok]).all(), (t, sid)
    return got


def test_surface_matches_the_oracle(plogp):
    from dataclasses import replace
    check_surface(plogp, wl.config1())
    check_surface(plogp, replace(wl.config1(), strategy_mask=wl.ALL_STRATEGIES, k_mode=1))
    check_surface(plogp, wl.config2(P_hi=70, n_m=37, n_s=13))                     # ragged tiles, all three ids
    check_surface(plogp, wl.config4(n_tables=5, P_hi=40, n_m=20, n_s=32), tables=[0, 2, 4])
    # a long, regular candidate list (every multiple of 4 B) and a list of process counts with gaps
    P = np.array([2, 3, 8, 9, 100, 1000], dtype=np.int32)
    w = replace(wl.config3(P_hi=1000, n_m=4, m_lo=1 << 10, m_hi=1 << 13, s_hi=1 << 12), P_list=P, strategy_mask=wl.ALL_STRATEGIES)
    got = check_surface(plogp, w)
    # the minimum of the surface over s is the prediction, the first s attaining it the reported best s
    import torch
    with plogp.Tables.from_workload(w) as tabs:
        pred = plogp.predict(tabs, w)
        torch.cuda.synchronize()
    for q, sid in enumerate((2, 5, 9)):
        low = np.nanmin(got[0, q], axis=-1)
        assert np.array_equal(low, pred.time[0, sid].cpu().numpy())
        first = np.nanargmin(got[0, q], axis=-1)
        assert np.array_equal(w.s_values()[first].astype(np.uint32), pred.best_s[0, q].cpu().numpy().view(np.uint32))


def check_fixed(plogp, w, s_fixed, tables=None):
    import torch
    from oracle import plogp_oracle as po
    ot = oracle_tables(w)
    with plogp.Tables.from_workload(w) as tabs:
        pred = plogp.predict(tabs, w)
        fixed, ratio = plogp.segment_sensitivity(tabs, w, s_fixed, pred)
        alone, none = plogp.segment_sensitivity(tabs, w, s_fixed)
        torch.cuda.synchronize()
    assert none is None and torch.equal(alone.view(torch.int64), fixed.view(torch.int64))
    fixed, ratio = fixed.cpu().numpy(), ratio.cpu().numpy()
    for t in (range(w.n_tables) if tables is None else tables):
        want = po.fixed_segment_grid(ot[t], w.strategy_mask, w.P_values(), w.m, s_fixed, w.k_mode)
        best = po.predict_grid(ot[t], w.strategy_mask, w.P_values(), w.m, oracle_sgrid(w), w.k_mode).time
        for q, sid in enumerate((2, 5, 9)):
            if not (w.strategy_mask >> sid) & 1:
                assert np.isnan(fixed[t, q]).all() and np.isnan(ratio[t, q]).all()
                continue
            assert (np.abs(fixed[t, q] - want[q]) <= RTOL * want[q]).all(), (t, sid)
            r = want[q] / best[sid]
            assert (np.abs(ratio[t, q] - r) <= 4 * RTOL * r).all(), (t, sid)


def test_fixed_segment_size_and_its_ratio_to_the_optimum(plogp):
    from dataclasses import replace
    for s_fixed in (8192, 4, 1 << 22, 100):   # the paper's 8 kB; the smallest size; one no message reaches; one off the grid
        check_fixed(plogp, replace(wl.config1(), strategy_mask=wl.ALL_STRATEGIES), s_fixed)
    check_fixed(plogp, wl.config2(P_hi=300, n_m=45, n_s=29), 8192)
    check_fixed(plogp, replace(wl.config2(P_hi=77, n_m=37, n_s=13), k_mode=1, strategy_mask=(1 << 5) | (7 << 10)), 1024)
    check_fixed(plogp, wl.config4(n_tables=6, P_hi=130), 8192, tables=[0, 3, 5])
    # a fixed size from the candidate list can never beat the search
    import torch
    w = wl.config4(n_tables=40)
    with plogp.Tables.from_workload(w) as tabs:
        pred = plogp.predict(tabs, w)
        s_fixed = int(w.s_list[20])
        fixed, ratio = plogp.segment_sensitivity(tabs, w, s_fixed, pred)
        torch.cuda.synchronize()
    fits = torch.as_tensor(w.m.astype(np.int64) >= s_fixed, device="cuda")
    assert bool((ratio[..., fits] >= 1.0).all()) and bool(torch.isfinite(fixed).all())


def test_refusals(plogp):
    import torch
    w = wl.config1()
    with plogp.Tables.from_workload(w) as tabs:
        g = plogp.GridArgs.from_workload(w)
        out = torch.zeros((1, 3, g.n_P, g.n_m), dtype=torch.float64, device="cuda")
        call = plogp.lib.plogp_segment_sensitivity
        assert call(tabs.handle, g.ref, 0, None, out.data_ptr(), None, None) == plogp.E_INVAL
        assert call(tabs.handle, g.ref, 6, None, out.data_ptr(), None, None) == plogp.E_INVAL       # not a multiple of the datatype
        assert call(tabs.handle, g.ref, 1 << 32, None, out.data_ptr(), None, None) == plogp.E_RANGE
        assert call(tabs.handle, g.ref, 8192, None, out.data_ptr(), out.data_ptr(), None) == plogp.E_INVAL   # ratio without predictions
        assert call(tabs.handle, g.ref, 8192, None, None, None, None) == plogp.E_INVAL
        assert plogp.lib.plogp_segment_surface(tabs.handle, g.ref, None, None) == plogp.E_INVAL
    assert plogp.lib.plogp_decision_boundaries(1, 4, 4, None, None, None) == plogp.E_INVAL
    assert plogp.lib.plogp_decision_boundaries(0, 4, 4, None, None, None) == plogp.OK


def test_decision_boundaries(plogp):
    import torch
    from oracle import plogp_oracle as po
    # message-size counts off and on a multiple of 8 (the second kind takes the 8-bytes-per-thread kernel)
    for w in (wl.config1(), wl.config2(P_hi=300, n_m=70, n_s=40), wl.config4(n_tables=7, P_hi=90, n_m=33),
              wl.config4(n_tables=5, P_hi=70, n_m=32), wl.config2(P_hi=130, n_m=8, n_s=20), wl.config4(n_tables=3)):
        with plogp.Tables.from_workload(w) as tabs:
            dec = plogp.select_best(tabs, w)
            b = plogp.decision_boundaries(dec)
            torch.cuda.synchronize()
        assert np.array_equal(b.cpu().numpy(), po.decision_boundaries(dec.strategy.cpu().numpy()))
        assert int(b.sum()) > 0        # these grids do have strategy changes
