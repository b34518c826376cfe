"""plogp_scatter_chain_static — the entry point for callers that may not allocate device memory
(its scan scratch is a fixed array inside the library) — against plogp_predict's Scatter Chain
plane and against the CPU oracle's, on calls in a row that share that array.  Collected last on
purpose."""
import numpy as np
import pytest

from paper_cs_0408034_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def both_ways(plogp, w):
    """Scatter Chain times of table 0 from the allocating path and from the static-scratch path."""
    import torch
    from dataclasses import replace
    w = replace(w, strategy_mask=1 << 11)
    with plogp.Tables(w.table_sizes(0), w.gaps[:1], w.latency[:1]) as tabs:
        ref = plogp.predict(tabs, w, want_best_s=False).time[0, 11].clone()
    d_sizes = torch.from_numpy(w.table_sizes(0).astype(np.int64)).cuda()
    d_gap = torch.from_numpy(np.ascontiguousarray(w.gaps[0])).cuda()
    d_m = torch.from_numpy(w.m.astype(np.int64)).cuda()
    got = plogp.scatter_chain_static(d_sizes, d_gap, float(w.latency[0]), w.P_lo, w.P_hi, d_m)
    torch.cuda.synchronize()
    return ref, got


def oracle_plane(w):
    """The oracle's Scatter Chain plane (Table 2, second row) for table 0."""
    from oracle import plogp_oracle as po
    tab = po.Table(w.table_sizes(0), w.gaps[0], w.latency[0])
    return po.predict_grid(tab, 1 << 11, w.P_values(), w.m, po.SGrid(lo=4, hi=4, step=4)).time[11]


def test_static_scratch_matches_predict_on_two_calls_in_a_row():
    import torch
    from paper_cs_0408034_b200 import plogp
    # first call: several P tiles and a ragged m tile; second call: a different, smaller shape,
    # so anything left in the shared array by the first call would show
    from dataclasses import replace
    # a first process count above 2 makes the first rows depend on terms that are never written out
    # (37 lies inside the first tile of 1024 terms, 2500 in the third)
    for w in (wl.config5(P_hi=5000, n_m=40), wl.config1(), wl.config5(P_hi=3333, n_m=64),
              replace(wl.config5(P_hi=4100, n_m=33), P_lo=37), replace(wl.config5(P_hi=2600, n_m=5), P_lo=2500)):
        ref, got = both_ways(plogp, w)
        assert got.shape == ref.shape
        rel = ((got - ref).abs() / ref).max().item()
        assert rel <= 1e-12, (w.name, rel)
        want = oracle_plane(w)
        rel = (np.abs(got.cpu().numpy() - want) / want).max()
        assert rel <= 1e-12, (w.name, rel)


def test_static_scratch_limits_are_refused():
    import torch
    from paper_cs_0408034_b200 import plogp
    d = torch.zeros(8, dtype=torch.int64, device="cuda")
    g = torch.zeros(8, dtype=torch.float64, device="cuda")
    out = torch.zeros(8, dtype=torch.float64, device="cuda")
    call = plogp.lib.plogp_scatter_chain_static
    assert call(8, d.data_ptr(), g.data_ptr(), 1.0, 2, 2 + 262144, d.data_ptr(), 1, out.data_ptr(), None) == plogp.E_RANGE
    assert call(8, d.data_ptr(), g.data_ptr(), 1.0, 262140, 2 + 262144, d.data_ptr(), 1, out.data_ptr(), None) == plogp.E_RANGE
    assert call(8, d.data_ptr(), g.data_ptr(), float("inf"), 2, 3, d.data_ptr(), 1, out.data_ptr(), None) == plogp.E_INVAL
    assert call(8, d.data_ptr(), g.data_ptr(), 1.0, 2, 3, d.data_ptr(), 257, out.data_ptr(), None) == plogp.E_RANGE
    assert call(2000, d.data_ptr(), g.data_ptr(), 1.0, 2, 3, d.data_ptr(), 1, out.data_ptr(), None) == plogp.E_RANGE
    assert call(8, None, g.data_ptr(), 1.0, 2, 3, d.data_ptr(), 1, out.data_ptr(), None) == plogp.E_INVAL
    assert call(8, d.data_ptr(), g.data_ptr(), 1.0, 1, 3, d.data_ptr(), 1, out.data_ptr(), None) == plogp.E_INVAL
