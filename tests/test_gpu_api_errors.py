"""Error paths of the C ABI: malformed tables and grids are refused on the host with a status code;
empty grids are no-ops.  Nothing here launches a kernel with bad arguments."""
import ctypes as C

import numpy as np
import pytest

from paper_cs_0408034_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plogp():
    import torch
    assert torch.cuda.is_available()
    from paper_cs_0408034_b200 import plogp as mod
    return mod


def load_status(plogp, sizes, gaps, lat, shared=1):
    sizes = np.ascontiguousarray(sizes, dtype=np.uint64)
    gaps = np.ascontiguousarray(gaps, dtype=np.float64)
    lat = np.ascontiguousarray(lat, dtype=np.float64)
    h = C.c_void_p()
    rc = plogp.lib.plogp_table_load(gaps.shape[0], gaps.shape[1], sizes.ctypes.data, shared, gaps.ctypes.data,
                                    lat.ctypes.data, C.byref(h))
    if rc == 0:
        plogp.lib.plogp_table_free(h)
    else:
        assert h.value is None
    return rc


def test_bad_tables(plogp):
    ok = ([4, 8, 16], [[1.0, 2.0, 3.0]], [1.0])
    assert load_status(plogp, *ok) == plogp.OK
    assert load_status(plogp, [4, 4, 16], ok[1], ok[2]) == plogp.E_INVAL      # sizes not increasing
    assert load_status(plogp, [4, 8, 16], [[1.0, np.nan, 3.0]], [1.0]) == plogp.E_INVAL
    assert load_status(plogp, [4, 8, 16], [[1.0, -2.0, 3.0]], [1.0]) == plogp.E_INVAL
    assert load_status(plogp, [4, 8, 16], ok[1], [np.inf]) == plogp.E_INVAL
    assert load_status(plogp, [4], [[1.0]], [1.0]) == plogp.E_INVAL             # fewer than two sizes
    assert load_status(plogp, [4, 8, 1 << 60], ok[1], ok[2]) == plogp.E_RANGE
    assert load_status(plogp, [4, 8, 16], [[1.0, 3.0, 2.5]], [1.0]) == plogp.E_RANGE   # falling last interval
    n = 1025
    assert load_status(plogp, np.arange(1, n + 1) * 4, [np.arange(n, dtype=np.float64)], [1.0]) == plogp.E_RANGE
    h = C.c_void_p()
    assert plogp.lib.plogp_table_load(1, 3, None, 1, None, None, C.byref(h)) == plogp.E_INVAL
    assert plogp.lib.plogp_table_free(None) == plogp.OK


def test_bad_grids_and_null_outputs(plogp):
    import torch
    w = wl.config1()
    with plogp.Tables.from_workload(w) as tabs:
        out = plogp.alloc_decision(1, 4, 2)

        def status(**kw):
            args = dict(m=[8, 16], P_lo=2, P_hi=5, s=[4, 8])
            args.update(kw)
            g = plogp.GridArgs(**args)
            return plogp.lib.plogp_select_best(tabs.handle, g.ref, out.strategy.data_ptr(), out.s_bytes.data_ptr(),
                                               out.time.data_ptr(), None)

        assert status() == plogp.OK
        assert status(P_lo=1) == plogp.E_INVAL
        assert status(P_lo=6, P_hi=5) == plogp.E_INVAL
        assert status(P_lo=(1 << 30) - 2, P_hi=(1 << 30) + 1, m=[4], s=[4]) == plogp.E_RANGE   # process counts above 2^30
        assert status(P=[2, (1 << 30) + 1], m=[4], s=[4]) == plogp.E_RANGE
        assert status(P=[2, 2, 3]) == plogp.E_INVAL
        assert status(P=[3, 1]) == plogp.E_INVAL
        assert status(m=[16, 8]) == plogp.E_INVAL
        assert status(m=[6, 16]) == plogp.E_INVAL          # not a multiple of the datatype
        assert status(m=[0, 16]) == plogp.E_INVAL
        assert status(s=[8, 4]) == plogp.E_INVAL
        assert status(s=[0, 4]) == plogp.E_INVAL
        assert status(s=None, s_lo=4, s_hi=16, s_step=0) == plogp.E_INVAL
        assert status(s=None, s_lo=4, s_hi=16, s_step=6) == plogp.E_INVAL
        assert status(dtype_bytes=0) == plogp.E_INVAL
        assert status(strategy_mask=1 << 13) == plogp.E_INVAL
        assert status(k_mode=2) == plogp.E_INVAL
        assert status(m=[8, 1 << 32]) == plogp.E_RANGE
        assert status(s=[4, 1 << 33]) == plogp.E_RANGE
        assert status(m=[8, 1 << 31], P_hi=1 << 23) == plogp.E_RANGE   # (P-1) m no longer exact in a double
        # segment list is ignored (not even validated) when no segmented strategy is enabled
        assert status(s=[8, 4], strategy_mask=0b1) == plogp.OK
        g = plogp.GridArgs([8, 16], P_lo=2, P_hi=5, s=[4, 8])
        assert plogp.lib.plogp_select_best(tabs.handle, g.ref, None, out.s_bytes.data_ptr(), out.time.data_ptr(), None) == plogp.E_INVAL
        assert plogp.lib.plogp_select_best(None, g.ref, out.strategy.data_ptr(), out.s_bytes.data_ptr(), out.time.data_ptr(), None) == plogp.E_INVAL
        assert plogp.lib.plogp_select_best(tabs.handle, None, out.strategy.data_ptr(), out.s_bytes.data_ptr(), out.time.data_ptr(), None) == plogp.E_INVAL
        assert plogp.lib.plogp_predict(tabs.handle, g.ref, None, None, None) == plogp.E_INVAL
        torch.cuda.synchronize()
        # a good call still works after all the refusals
        assert status() == plogp.OK
        torch.cuda.synchronize()


def test_empty_grids_are_no_ops(plogp):
    import torch
    w = wl.config1()
    with plogp.Tables.from_workload(w) as tabs:
        out = plogp.alloc_decision(1, 4, 2)
        for g in (plogp.GridArgs([], P_lo=2, P_hi=5, s=[4]),
                  plogp.GridArgs([8, 16], P=[], s=[4]),
                  plogp.GridArgs([8, 16], P_lo=2, P_hi=5, s=[4], strategy_mask=0)):
            plogp.select_best(tabs, g, out=out)
        torch.cuda.synchronize()
        assert (out.strategy == 255).all() and torch.isnan(out.time).all()
        # no candidate list at all: segmented strategies fall back to the whole message
        g = plogp.GridArgs([8, 16], P_lo=2, P_hi=5, s=[], strategy_mask=(1 << 5) | (1 << 3))
        dec = plogp.select_best(tabs, g)
        torch.cuda.synchronize()
        assert (dec.strategy[0, 0] == 3).all() and (dec.s_bytes[0, 0] == 0).all()
        g = plogp.GridArgs([8, 16], P_lo=2, P_hi=5, s=[], strategy_mask=1 << 5)
        pred = plogp.predict(tabs, g)
        torch.cuda.synchronize()
        assert pred.best_s[0, 1, :, 0].tolist() == [8] * 4 and pred.best_s[0, 1, :, 1].tolist() == [16] * 4


def test_fp64_rate_probe(plogp):
    r = plogp.fp64_fma_rate(5.0)
    assert 1e12 < r < 1e14
    assert plogp.lib.plogp_fp64_fma_rate(-1.0) < 0
