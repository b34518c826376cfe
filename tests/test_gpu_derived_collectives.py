"""plogp_select_best_collective (Gather, Reduce, Barrier — the collectives the paper names without printing models)
through the C ABI against the CPU oracle's derived models, under the acceptance rule of tests/parity.py."""
import numpy as np
import pytest

from paper_cs_0408034_b200 import workloads as wl
from parity import TIE_MARGIN, TIME_RTOL, _valid_s, oracle_sgrid, oracle_tables

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plogp():
    import torch
    assert torch.cuda.is_available()
    from paper_cs_0408034_b200 import plogp as mod
    return mod


def oracle_mask(collective, mask):
    """Grid mask (bits of the mirrored printed ids) -> oracle mask (bits of the derived ids)."""
    from oracle import plogp_oracle as po
    table = po.MIRROR_OF if collective != po.BARRIER else po.BARRIER_SHAPE_OF
    lo = po.DERIVED_FIRST_ID[collective]
    hi = {po.GATHER: 16, po.REDUCE: 23, po.BARRIER: 27}[collective]
    return sum(1 << d for d in range(lo, hi) if (mask >> table[d]) & 1)


def check(plogp, w, collective, tables=None):
    import torch
    from oracle import plogp_oracle as po
    ot = oracle_tables(w)
    with plogp.Tables.from_workload(w) as tabs:
        dec = plogp.select_best_collective(tabs, w, collective)
        torch.cuda.synchronize()
    g_id, g_s, g_t = dec.strategy.cpu().numpy(), dec.s_bytes.cpu().numpy().view(np.uint32), dec.time.cpu().numpy()
    omask = oracle_mask(collective, w.strategy_mask)
    ms = w.m if collective != po.BARRIER else w.m[:1]
    n = 0
    for t in (range(w.n_tables) if tables is None else tables):
        o = po.decide_grid(ot[t], collective, omask, w.P_values(), ms, oracle_sgrid(w), w.k_mode)
        gi, gs, gt = (x[t].reshape(o.strategy.shape) for x in (g_id, g_s, g_t))
        if omask == 0:
            assert (gi == 255).all()
            continue
        same = (gi == o.strategy) & (gs == o.s)
        assert (np.abs(gt[same] - o.time[same]) <= TIME_RTOL * o.time[same]).all(), (t, collective)
        for ip, im in zip(*np.nonzero(~same)):   # another pick: only inside the tie margin, with the oracle's time for it
            P, m = int(w.P_values()[ip]), int(ms[im])
            gid, s = int(gi[ip, im]), int(gs[ip, im])
            assert (omask >> gid) & 1, (t, P, m, gid)
            if gid in (17, 19, 22):
                assert _valid_s(w, m, s)
            else:
                assert s == 0
            alt = po.model(ot[t], gid, P, m, s, w.k_mode)
            assert (alt - o.time[ip, im]) / o.time[ip, im] <= TIE_MARGIN, (t, P, m, gid, s)
            assert abs(gt[ip, im] - alt) <= TIME_RTOL * alt
        n += gi.size
    return n


def test_gather_reduce_barrier_match_the_oracle(plogp):
    from dataclasses import replace
    from oracle import plogp_oracle as po
    grids = [replace(wl.config1(), strategy_mask=wl.ALL_STRATEGIES),
             wl.config2(P_hi=300, n_m=45, n_s=29),
             replace(wl.config2(P_hi=77, n_m=37, n_s=13), k_mode=1),
             replace(wl.config5(P_hi=3000, n_m=40), strategy_mask=wl.ALL_STRATEGIES),        # several P tiles in the Gather
             replace(wl.config3(P_hi=300, n_m=6, m_lo=1 << 10, m_hi=1 << 15, s_hi=1 << 13), strategy_mask=wl.ALL_STRATEGIES)]  # long lists
    for w in grids:
        for coll in (po.GATHER, po.REDUCE, po.BARRIER):
            assert check(plogp, w, coll) > 0
    w = wl.config4(n_tables=6, P_hi=200)
    for coll in (po.GATHER, po.REDUCE, po.BARRIER):
        assert check(plogp, w, coll, tables=[0, 3, 5]) > 0
    # the lower-envelope search serves the Reduce as well
    assert check(plogp, replace(wl.config2(P_hi=300, n_m=45, n_s=29), search_mode=1), po.REDUCE) > 0


def test_subsets_of_strategies_and_relabelled_ids(plogp):
    from dataclasses import replace
    from oracle import plogp_oracle as po
    base = wl.config2(P_hi=120, n_m=30, n_s=20)
    for mask in (1 << 11, (1 << 10) | (1 << 12), 1 << 5, (1 << 0) | (1 << 7), (1 << 2) | (1 << 9), (1 << 3) | (1 << 6), (1 << 1) | (1 << 4) | (1 << 8)):
        for coll in (po.GATHER, po.REDUCE, po.BARRIER):
            check(plogp, replace(base, strategy_mask=mask), coll)   # collectives with nothing enabled stay untouched (255)


def test_refusals(plogp):
    import torch
    w = wl.config1()
    with plogp.Tables.from_workload(w) as tabs:
        g = plogp.GridArgs.from_workload(w)
        out = plogp.alloc_decision(1, g.n_P, g.n_m)
        call = plogp.lib.plogp_select_best_collective
        args = (out.strategy.data_ptr(), out.s_bytes.data_ptr(), out.time.data_ptr(), None)
        assert call(tabs.handle, g.ref, 0, *args) == plogp.E_INVAL      # Broadcast and Scatter are plogp_select_best's
        assert call(tabs.handle, g.ref, 7, *args) == plogp.E_INVAL
        assert call(tabs.handle, g.ref, plogp.GATHER, None, None, None, None) == plogp.E_INVAL
        assert call(None, g.ref, plogp.GATHER, *args) == plogp.E_INVAL
