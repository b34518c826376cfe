"""GPU results through the C ABI against the CPU oracle, element by element, on seeded workloads
shaped like the five benchmark configurations (reduced where the oracle would take too long) plus
edge cases.  Tolerances: see tests/parity.py."""
import numpy as np
import pytest

from paper_cs_0408034_b200 import workloads as wl
from parity import check_decision, check_decision_cells, check_prediction, oracle_tables

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plogp():
    import torch
    assert torch.cuda.is_available()
    from paper_cs_0408034_b200 import plogp as mod
    return mod


def run_both(plogp, w, **sub):
    import torch
    ot = oracle_tables(w)
    with plogp.Tables.from_workload(w) as tabs:
        dec = plogp.select_best(tabs, w)
        pred = plogp.predict(tabs, w)
        torch.cuda.synchronize()
        n = check_decision(w, ot, dec, **sub) + check_prediction(w, ot, pred, **sub)
    assert n > 0
    return dec, pred


def test_config1_full(plogp):
    run_both(plogp, wl.config1())


def test_config1_all_strategies_and_floor_mode(plogp):
    from dataclasses import replace
    w = replace(wl.config1(), strategy_mask=wl.ALL_STRATEGIES)
    run_both(plogp, w)
    run_both(plogp, replace(w, k_mode=1))


def test_config2_full_size(plogp):
    # 1023 x 256 cells x 13 strategies, 64 candidates: the oracle needs a few seconds
    run_both(plogp, wl.config2())


def test_config2_ragged_tiles(plogp):
    # n_m = 37 (one full tile + ragged tail), n_P = 77 (ragged pass), 13 candidates
    run_both(plogp, wl.config2(P_hi=78, n_m=37, n_s=13))


def test_config3_reduced_goes_through_the_sweep_kernel(plogp):
    # candidates = every multiple of 4 up to 64 KB (16384 > inline limit): chunks, several P tiles' worth of lanes
    w = wl.config3(P_hi=300, n_m=10, m_lo=4 << 10, m_hi=1 << 18, s_hi=1 << 16)
    run_both(plogp, w)


def test_config3_sweep_with_all_segmented_strategies(plogp):
    from dataclasses import replace
    w = replace(wl.config3(P_hi=2200, n_m=5, m_lo=1 << 10, m_hi=1 << 15, s_hi=1 << 13), strategy_mask=wl.ALL_STRATEGIES)
    run_both(plogp, w, p_idx=np.r_[0:40, 1000:1040, 2040:2060, 2190:2199])
    for mask in (1 << 2, 1 << 9, (1 << 2) | (1 << 9), (1 << 5) | (1 << 9)):
        run_both(plogp, replace(w, strategy_mask=mask, P_hi=130))


def test_config4_reduced_batch(plogp):
    w = wl.config4(n_tables=6)
    run_both(plogp, w, tables=[0, 3, 5], p_idx=np.r_[0:70, 250:260, 500:511])


def test_config5_reduced_long_scan(plogp):
    # P up to 9000: several P tiles, exercises the tile-sum / tile-scan carry of the Scatter Chain
    run_both(plogp, wl.config5(P_hi=9000, n_m=40))


def test_config5_full_size_sampled_rows(plogp):
    import torch
    w = wl.config5()
    ot = oracle_tables(w)
    with plogp.Tables.from_workload(w) as tabs:
        dec = plogp.select_best(tabs, w)
        pred = plogp.predict(tabs, w, want_best_s=False)
        torch.cuda.synchronize()
        p_idx = np.unique(np.r_[0:64, 4090:4100, 32760:32775, 65500:65535, np.arange(0, 65535, 997)])
        m_idx = np.array([0, 1, 31, 32, 63])
        check_decision(w, ot, dec, p_idx=p_idx, m_idx=m_idx)
        check_prediction(w, ot, pred, p_idx=p_idx, m_idx=m_idx)


def test_explicit_P_list_with_gaps(plogp):
    import torch
    w = wl.config1()
    P = np.array([2, 3, 4, 8, 9, 16, 17, 31, 32, 33, 50, 400, 1000], dtype=np.int32)
    g = plogp.GridArgs(w.m, P=P, s=w.s_list, strategy_mask=wl.ALL_STRATEGIES)
    from oracle import plogp_oracle as po
    ot = oracle_tables(w)[0]
    with plogp.Tables.from_workload(w) as tabs:
        pred = plogp.predict(tabs, g)
        torch.cuda.synchronize()
    o = po.predict_grid(ot, wl.ALL_STRATEGIES, P, w.m, po.SGrid(w.s_list))
    got = pred.time[0].cpu().numpy()
    assert np.max(np.abs(got - o.time) / o.time) <= 1e-12
    assert (pred.best_s[0].cpu().numpy().view(np.uint32) == o.best_s).all()


def test_deterministic_across_runs(plogp):
    import torch
    w = wl.config2(P_hi=300, n_m=70, n_s=40)
    with plogp.Tables.from_workload(w) as tabs:
        a = plogp.select_best(tabs, w)
        b = plogp.select_best(tabs, w)
        torch.cuda.synchronize()
    assert torch.equal(a.strategy, b.strategy) and torch.equal(a.s_bytes, b.s_bytes)
    assert torch.equal(a.time.view(torch.int64), b.time.view(torch.int64))


def test_single_cell_and_two_breakpoints(plogp):
    import torch
    from oracle import plogp_oracle as po
    sizes = np.array([4, 1024], dtype=np.uint64)
    gaps = np.array([[2.0, 12.0]])
    with plogp.Tables(sizes, gaps, np.array([3.0])) as tabs:
        g = plogp.GridArgs([512], P_lo=7, P_hi=7, s=[4, 64, 512, 1024])
        pred = plogp.predict(tabs, g)
        dec = plogp.select_best(tabs, g)
        torch.cuda.synchronize()
    t = po.Table(sizes, gaps[0], 3.0)
    o = po.predict_grid(t, wl.ALL_STRATEGIES, [7], [512], po.SGrid([4, 64, 512, 1024]))
    np.testing.assert_allclose(pred.time[0, :, 0, 0].cpu().numpy(), o.time[:, 0, 0], rtol=1e-12)
    od = po.select_grid(wl.ALL_STRATEGIES, o)
    assert dec.strategy[0, :, 0, 0].tolist() == od.strategy[:, 0, 0].tolist()


def test_config4_full_size_sampled_tables(plogp):
    """The benchmark's launch configuration (4096 tables, decide_kernel + scatter_kernel); whole decision
    tables of sampled networks, first / middle / last, are compared with the oracle."""
    import torch
    w = wl.config4()
    ot = {t: None for t in (0, 1, 777, 2048, 4095)}
    from oracle import plogp_oracle as po
    for t in ot:
        ot[t] = po.Table(w.table_sizes(t), w.gaps[t], w.latency[t])
    with plogp.Tables.from_workload(w) as tabs:
        dec = plogp.select_best(tabs, w)
        torch.cuda.synchronize()
        n = check_decision(w, ot, dec, tables=list(ot))
        # a seeded sample of 2e5 (table, P, m) cells over all 4096 tables, each re-decided by the oracle
        k = 200000
        c = np.arange(k)
        t_idx = (wl.uniform(w.seed, 7_000_000 + c) * w.n_tables).astype(np.int64)
        p_idx = (wl.uniform(w.seed, 8_000_000 + c) * w.n_P).astype(np.int64)
        m_idx = (wl.uniform(w.seed, 9_000_000 + c) * w.n_m).astype(np.int64)
        assert len(np.unique(t_idx)) > 4000
        assert check_decision_cells(w, dec, t_idx, p_idx, m_idx) == 2 * k
    assert n == len(ot) * 2 * w.n_P * w.n_m
    # every cell of every table was written, with an eligible id
    assert int((dec.strategy[:, 0] > 9).sum()) == 0 and int(((dec.strategy[:, 1] < 10) | (dec.strategy[:, 1] > 12)).sum()) == 0
    assert bool(torch.isfinite(dec.time).all())


def test_config3_full_size_sampled_cells(plogp):
    """The exhaustive sweep at full size (262144 candidates, P up to 4096) in the benchmark's launch
    configuration; the oracle re-searches 64 x 32 = 2048 sampled (P, m) cells (tile edges of the sweep
    kernel's P tiles and warps, plus a seeded spread), predictions and decisions."""
    import torch
    w = wl.config3()
    ot = oracle_tables(w)
    edges = [0, 1, 2, 30, 31, 32, 255, 256, 257, 1000, 2047, 2048, 2049, 3000, 4093, 4094]
    spread = (wl.uniform(w.seed, 5000 + np.arange(48)) * w.n_P).astype(np.int64)
    p_idx = np.unique(np.r_[edges, spread])
    m_idx = np.unique(np.r_[[0, 1, 40, 63, 64, 90, 126, 127], (wl.uniform(w.seed, 6000 + np.arange(24)) * w.n_m).astype(np.int64)])
    with plogp.Tables.from_workload(w) as tabs:
        pred = plogp.predict(tabs, w)
        dec = plogp.select_best(tabs, w)
        torch.cuda.synchronize()
        n = check_prediction(w, ot, pred, p_idx=p_idx, m_idx=m_idx) + check_decision(w, ot, dec, p_idx=p_idx, m_idx=m_idx)
    assert n >= 2000
    assert bool(torch.isnan(pred.time[0, [0, 1, 3, 4, 6, 7, 8, 9, 10, 11, 12]]).all())


def test_select_best_with_explicit_P_list_and_per_table_sizes(plogp):
    """Decision kernels on a process-count list with gaps (Scatter Chain terms span several j) and on
    tables that do not share their size lists, under the full acceptance rule."""
    sizes = np.stack([wl.log_spaced_multiples(4, 1 << 20, 16), wl.log_spaced_multiples(8, 1 << 22, 16),
                      wl.log_spaced_multiples(4, 1 << 18, 16)])
    gaps = np.stack([wl.noisy_monotone_gaps(sizes[t], 2.0 + t, 0.004 * (t + 1), 0.05, 77 + t) for t in range(3)])
    lat = np.array([3.0, 11.0, 0.5])
    P = np.array([2, 3, 5, 8, 13, 21, 34, 55, 89, 144, 233, 377, 610, 987], dtype=np.int32)
    w = wl.Workload("explicit_P_list", sizes, gaps, lat, int(P[0]), int(P[-1]), wl.log_spaced_multiples(4, 1 << 21, 21),
                    s_list=wl.log_spaced_multiples(4, 1 << 19, 11), P_list=P)
    run_both(plogp, w)
    from dataclasses import replace
    run_both(plogp, replace(w, k_mode=1))


def test_host_output_entry_point_matches_device_outputs(plogp):
    """plogp_select_best_host streams the decision table to host arrays in batches (here 3 batches of
    tables through the two staging sets); it must equal plogp_select_best bit for bit."""
    import torch
    w = wl.config4(n_tables=700)
    with plogp.Tables.from_workload(w) as tabs:
        dev = plogp.select_best(tabs, w)
        host = plogp.select_best_host(tabs, w)
        host2 = plogp.select_best_host(tabs, w)   # staging sets and events are reused
        torch.cuda.synchronize()
    for h in (host, host2):
        assert torch.equal(h.strategy, dev.strategy.cpu())
        assert torch.equal(h.s_bytes, dev.s_bytes.cpu())
        assert torch.equal(h.time.view(torch.int64), dev.time.cpu().view(torch.int64))
    small = wl.config1()
    with plogp.Tables.from_workload(small) as tabs:
        a, b = plogp.select_best(tabs, small), plogp.select_best_host(tabs, small)
    assert torch.equal(b.strategy, a.strategy.cpu()) and torch.equal(b.time.view(torch.int64), a.time.cpu().view(torch.int64))


def test_many_tables_take_the_gap_prepass(plogp):
    """Enough tables for the host to run gaps_kernel in front of the lane <-> P kernels (g(1), g(s), g(m) read from
    its rows instead of interpolated in every CTA), with a last group of message sizes that is not full, in both
    segment-count modes; three tables are compared with the oracle."""
    from dataclasses import replace
    base = wl.config4(n_tables=320, P_hi=300, n_m=34, n_s=20, seed_offset=11)
    for k_mode in (0, 1):
        w = replace(base, k_mode=k_mode)
        ot = oracle_tables(w)
        import torch
        with plogp.Tables.from_workload(w) as tabs:
            dec = plogp.select_best(tabs, w)
            pred = plogp.predict(tabs, w)
            torch.cuda.synchronize()
            n = check_decision(w, ot, dec, tables=[0, 157, 319]) + check_prediction(w, ot, pred, tables=[0, 157, 319])
        assert n > 0


def test_repeated_call_can_be_replayed_from_a_cuda_graph(plogp):
    """With its plan cached a call only launches kernels on the caller's stream, so it can be captured into a CUDA
    graph and replayed; the replay must reproduce the direct call bit for bit (decision kernel and Scatter kernels)."""
    import torch
    for w in (wl.config1(), wl.config5(P_hi=3000, n_m=40)):
        with plogp.Tables.from_workload(w) as tabs:
            dec = plogp.select_best(tabs, w)  # builds the plan, allocates scratch
            torch.cuda.synchronize()
            st = torch.cuda.Stream()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(st):
                plogp.select_best(tabs, w, out=dec, stream=st)
                st.synchronize()
                with torch.cuda.graph(graph, stream=st):
                    plogp.select_best(tabs, w, out=dec, stream=st)
            for t in (dec.strategy, dec.s_bytes, dec.time):
                t.zero_()
            plogp.select_best(tabs, w, out=dec)
            torch.cuda.synchronize()
            ref = (dec.strategy.clone(), dec.s_bytes.clone(), dec.time.clone())
            for t in (dec.strategy, dec.s_bytes, dec.time):
                t.zero_()
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(dec.strategy, ref[0]) and torch.equal(dec.s_bytes, ref[1])
            assert torch.equal(dec.time.view(torch.int64), ref[2].view(torch.int64))
            del graph


def test_randomised_grids_against_the_oracle(plogp):
    """Forty seeded random grids (1-5 tables; ranges, sub-ranges and lists of process counts that end inside, at and
    past a tile of 256; 1-40 message sizes; 1-64 candidates, some grids with message sizes below every candidate;
    random strategy masks; both segment-count modes and both search modes): decision table and predictions of every
    cell against the oracle."""
    from dataclasses import replace
    import torch
    rng = np.random.default_rng(408034)
    for case in range(40):
        nt = int(rng.integers(1, 6))
        P_hi = int(rng.choice([3, 9, 33, 70, 257, 300, 513, 600]))
        base = wl.config4(n_tables=nt, P_hi=P_hi, n_m=int(rng.integers(1, 41)), n_s=int(rng.integers(1, 65)), seed_offset=1000 + case)
        mask = wl.ALL_STRATEGIES if rng.random() < 0.3 else int(rng.integers(1, 1 << 13))
        kw = dict(strategy_mask=mask, k_mode=int(rng.integers(0, 2)), search_mode=int(rng.integers(0, 2)))
        pick = rng.random()
        if pick < 0.3:
            Ps = np.unique(rng.integers(2, P_hi + 1, size=int(rng.integers(1, 30)))).astype(np.int32)
            kw.update(P_list=Ps, P_lo=int(Ps[0]), P_hi=int(Ps[-1]))
        elif pick < 0.6:
            kw.update(P_lo=int(rng.integers(2, P_hi + 1)))
        if rng.random() < 0.2:
            kw.update(s_list=wl.log_spaced_multiples(1 << 10, 1 << 20, len(base.s_list)))
        w = replace(base, **kw)
        ot = oracle_tables(w)
        with plogp.Tables.from_workload(w) as tabs:
            dec = plogp.select_best(tabs, w)
            pred = plogp.predict(tabs, w)
            torch.cuda.synchronize()
            assert check_decision(w, ot, dec) + check_prediction(w, ot, pred) > 0, case


def test_sweep_kernel_with_several_tables(plogp):
    """Long candidate list (512 multiples of 4 B) on three independent tables: the sweep kernel's table
    dimension and the reduction of its partial minima per table."""
    from dataclasses import replace
    base = wl.config4(n_tables=3, P_hi=70, n_m=9)
    w = replace(base, s_list=None, s_lo=4, s_hi=2048, s_step=4)
    run_both(plogp, w)


def test_exact_ties_go_to_smallest_segment_and_lowest_id(plogp):
    """A flat table (g = 1 everywhere, L = 2) makes every model an exact small integer, so ties between
    candidates with the same segment count and between strategies are exact on both sides: the GPU must
    then reproduce the oracle's picks bit for bit (smallest s, lowest id), whatever order it sweeps in."""
    import torch
    from oracle import plogp_oracle as po
    sizes = np.array([4, 64, 1024, 1 << 20], dtype=np.uint64)
    gaps = np.ones((1, 4))
    lat = np.array([2.0])
    m = np.array([8, 100, 1000, 4096, 10000, 65536, 100000], dtype=np.uint64)
    P = np.arange(2, 140, dtype=np.int32)
    tab = po.Table(sizes, gaps[0], 2.0)
    for s_kw, sg in ((dict(s=wl.log_spaced_multiples(4, 1 << 16, 40)), po.SGrid(wl.log_spaced_multiples(4, 1 << 16, 40))),
                     (dict(s=None, s_lo=4, s_hi=4096, s_step=4), po.SGrid(lo=4, hi=4096, step=4))):
        g = plogp.GridArgs(m, P=P, **s_kw)
        with plogp.Tables(sizes, gaps, lat) as tabs:
            dec = plogp.select_best(tabs, g)
            pred = plogp.predict(tabs, g)
            torch.cuda.synchronize()
        o = po.predict_grid(tab, wl.ALL_STRATEGIES, P, m, sg)
        od = po.select_grid(wl.ALL_STRATEGIES, o)
        assert np.array_equal(pred.time[0].cpu().numpy(), o.time)
        assert np.array_equal(pred.best_s[0].cpu().numpy().view(np.uint32), o.best_s)
        assert np.array_equal(dec.strategy[0].cpu().numpy(), od.strategy)
        assert np.array_equal(dec.s_bytes[0].cpu().numpy().view(np.uint32), od.s)
        assert np.array_equal(dec.time[0].cpu().numpy(), od.time)


def test_table_update_replaces_contents_in_place(plogp):
    import torch
    a, b = wl.config4(n_tables=5, P_hi=40, n_m=12), wl.config4(n_tables=5, P_hi=40, n_m=12, seed_offset=9)
    with plogp.Tables.from_workload(a) as tabs:
        first = plogp.select_best(tabs, a)
        tabs.update(b.sizes, b.gaps, b.latency)
        second = plogp.select_best(tabs, b)
        torch.cuda.synchronize()
        check_decision(b, oracle_tables(b), second)
        assert not torch.equal(first.time, second.time)
        bad = b.gaps.copy()
        bad[2, 3] = float("nan")
        with pytest.raises(plogp.PlogpError):
            tabs.update(b.sizes, bad, b.latency)
        again = plogp.select_best(tabs, b)       # device tables untouched by the refused update
        torch.cuda.synchronize()
        assert torch.equal(again.time.view(torch.int64), second.time.view(torch.int64))


# ---- short candidate lists (decision kernel) with every combination of segmented strategies ----

@pytest.mark.parametrize("ids", [(2,), (9,), (5,), (2, 5), (5, 9), (2, 9), (0, 2, 7), (3, 5, 6, 8), (1, 4, 9), (2, 5, 9)])
def test_short_lists_with_subsets_of_strategies(plogp, ids):
    """<= 64 candidates, so the Broadcast half goes through the short-list decision kernel; masks with one,
    two or three segmented strategies, with and without unsegmented competitors, in both k modes.  The
    Scatter strategies stay enabled so that the Scatter half runs beside it."""
    from dataclasses import replace
    mask = sum(1 << i for i in ids) | (7 << 10)
    w = replace(wl.config2(P_hi=300, n_m=45, n_s=29), strategy_mask=mask)
    run_both(plogp, w)
    run_both(plogp, replace(w, k_mode=1, P_hi=70))
    run_both(plogp, replace(w, strategy_mask=mask & 0x3FF, P_hi=40))   # Broadcast strategies only


def test_floor_mode_on_the_sweep_kernel_and_on_several_tables(plogp):
    """k = floor(m/s) as Section 3.1 prints it, on a long candidate list (sweep kernel, all three segmented
    strategies) and on a three-table short-list grid."""
    from dataclasses import replace
    long_list = replace(wl.config3(P_hi=700, n_m=6, m_lo=1 << 10, m_hi=1 << 16, s_hi=1 << 14),
                        strategy_mask=wl.ALL_STRATEGIES, k_mode=1)
    run_both(plogp, long_list, p_idx=np.r_[0:50, 250:270, 500:520, 690:699])
    run_both(plogp, replace(wl.config4(n_tables=3, P_hi=200, n_m=40), k_mode=1))


def test_predict_at_the_batched_launch_shape(plogp):
    """plogp_predict on all 4096 tables of the batched workload (the launch shape the benchmark times):
    sampled tables and process-count rows of the prediction planes against the oracle."""
    import torch
    w = wl.config4()
    tabs_idx = [0, 1365, 2730, 4095]
    ot = {t: None for t in tabs_idx}
    from oracle import plogp_oracle as po
    for t in ot:
        ot[t] = po.Table(w.table_sizes(t), w.gaps[t], w.latency[t])
    with plogp.Tables.from_workload(w) as tabs:
        pred = plogp.predict(tabs, w)
        torch.cuda.synchronize()
        n = check_prediction(w, ot, pred, tables=tabs_idx, p_idx=np.r_[0:40, 250:262, 480:511])
        assert n > 0
        assert bool(torch.isfinite(pred.time).all())
    del pred
    torch.cuda.empty_cache()


def test_scatter_chain_with_a_far_first_process_count_and_wide_gaps(plogp):
    """Scatter Chain terms that span thousands of j (a contiguous range that starts far above 2, a
    process-count list with wide gaps): the library sums them per table interval in closed form, the oracle
    term by term."""
    from dataclasses import replace
    base = wl.config5(P_hi=300, n_m=37)
    run_both(plogp, replace(base, P_lo=100000, P_hi=100300))
    P = np.array([2, 3, 5000, 5001, 70000, 70001, 262144, 1000000], dtype=np.int32)
    run_both(plogp, replace(base, P_lo=2, P_hi=int(P[-1]), P_list=P))
    # the same through the general kernel (Broadcast strategies enabled as well)
    run_both(plogp, replace(wl.config2(P_hi=40, n_m=20, n_s=9), P_lo=3000, P_hi=3040))


# ---- search_mode 1: the segment-size search by lower envelope (same results as the exhaustive search) ----

def _envelope(w):
    from dataclasses import replace
    return replace(w, search_mode=1)


def test_envelope_search_on_short_and_long_candidate_lists(plogp):
    from dataclasses import replace
    run_both(plogp, _envelope(wl.config1()))
    run_both(plogp, _envelope(replace(wl.config1(), strategy_mask=wl.ALL_STRATEGIES, k_mode=1)))
    run_both(plogp, _envelope(wl.config2(P_hi=300, n_m=45, n_s=29)))
    run_both(plogp, _envelope(wl.config4(n_tables=6)), tables=[0, 3, 5], p_idx=np.r_[0:70, 250:260, 500:511])
    # long lists: every multiple of 4 B (16384 candidates), all three segmented strategies, both k modes
    w = replace(wl.config3(P_hi=700, n_m=6, m_lo=1 << 10, m_hi=1 << 16, s_hi=1 << 14), strategy_mask=wl.ALL_STRATEGIES)
    run_both(plogp, _envelope(w), p_idx=np.r_[0:50, 250:270, 500:520, 690:699])
    run_both(plogp, _envelope(replace(w, k_mode=1)), p_idx=np.r_[0:50, 250:270, 500:520, 690:699])
    for mask in (1 << 2, 1 << 5, 1 << 9, (1 << 2) | (1 << 9), (1 << 5) | (1 << 9)):
        run_both(plogp, _envelope(replace(w, strategy_mask=mask, P_hi=130)))


def test_envelope_search_with_more_representatives_than_fit_in_shared_memory(plogp):
    """m = 48 MB with every multiple of 4 B up to 1 MB as candidates: more than 6144 distinct segment counts, so
    the list of representatives goes through shared memory in several windows."""
    from dataclasses import replace
    w = replace(wl.config3(P_hi=600, n_m=2, m_lo=48 << 20, m_hi=49 << 20), search_mode=1)
    k = -(-int(w.m[0]) // np.arange(4, (1 << 20) + 1, 4))
    assert len(np.unique(k)) > 6144
    run_both(plogp, w, p_idx=np.r_[0:40, 100:110, 300:340, 590:599])


def test_envelope_search_on_a_table_with_a_dip_takes_the_exhaustive_search(plogp):
    """A table whose gap decreases somewhere does not qualify for the envelope search; the call must still
    return the exhaustive result."""
    import torch
    w = wl.config2(P_hi=120, n_m=30, n_s=20)
    gaps = w.gaps.copy()
    gaps[0, 7] = gaps[0, 6] * 0.9   # a dip in the middle; the last interval still rises
    from dataclasses import replace
    run_both(plogp, replace(w, gaps=gaps, search_mode=1))


def test_envelope_search_reproduces_exact_ties(plogp):
    """The flat table of the exact-tie test: with search_mode 1 the picks must equal the exhaustive ones bit for bit."""
    import torch
    sizes = np.array([4, 64, 1024, 1 << 20], dtype=np.uint64)
    gaps = np.ones((1, 4))
    lat = np.array([2.0])
    m = np.array([8, 100, 1000, 4096, 10000, 65536, 100000], dtype=np.uint64)
    P = np.arange(2, 140, dtype=np.int32)
    for s_kw in (dict(s=wl.log_spaced_multiples(4, 1 << 16, 40)), dict(s=None, s_lo=4, s_hi=4096, s_step=4)):
        with plogp.Tables(sizes, gaps, lat) as tabs:
            a = plogp.select_best(tabs, plogp.GridArgs(m, P=P, **s_kw))
            b = plogp.select_best(tabs, plogp.GridArgs(m, P=P, search_mode=1, **s_kw))
            pa = plogp.predict(tabs, plogp.GridArgs(m, P=P, **s_kw))
            pb = plogp.predict(tabs, plogp.GridArgs(m, P=P, search_mode=1, **s_kw))
            torch.cuda.synchronize()
        assert torch.equal(a.strategy, b.strategy) and torch.equal(a.s_bytes, b.s_bytes)
        assert torch.equal(a.time.view(torch.int64), b.time.view(torch.int64))
        assert torch.equal(pa.best_s, pb.best_s) and torch.equal(pa.time.view(torch.int64), pb.time.view(torch.int64))


def test_envelope_search_at_full_size(plogp):
    """The exhaustive-sweep configuration (262144 candidates, P up to 4096) and the batched one (4096 tables)
    through the envelope search: sampled cells against the oracle, everything else against the exhaustive path."""
    import torch
    w = wl.config3()
    ot = oracle_tables(w)
    p_idx = np.unique(np.r_[[0, 1, 2, 63, 64, 65, 255, 256, 2047, 2048, 4093, 4094], (wl.uniform(w.seed, 5100 + np.arange(30)) * w.n_P).astype(np.int64)])
    m_idx = np.unique(np.r_[[0, 1, 64, 127], (wl.uniform(w.seed, 6100 + np.arange(12)) * w.n_m).astype(np.int64)])
    with plogp.Tables.from_workload(w) as tabs:
        ex = plogp.select_best(tabs, w)
        env = plogp.select_best(tabs, _envelope(w))
        torch.cuda.synchronize()
        assert check_decision(w, ot, env, p_idx=p_idx, m_idx=m_idx) > 0
    same = (ex.strategy == env.strategy) & (ex.s_bytes == env.s_bytes)
    # wherever the picks differ the two times must agree to 1e-9 (ties inside the margin)
    rel = ((ex.time - env.time).abs() / ex.time)[:, 0]
    assert float(rel.max()) <= 1e-9
    assert float(same[:, 0].float().mean()) > 0.999
    w4 = wl.config4()
    with plogp.Tables.from_workload(w4) as tabs:
        env = plogp.select_best(tabs, _envelope(w4))
        torch.cuda.synchronize()
        k = 20000
        c = np.arange(k)
        t_idx = (wl.uniform(w4.seed, 7_500_000 + c) * w4.n_tables).astype(np.int64)
        pi = (wl.uniform(w4.seed, 8_500_000 + c) * w4.n_P).astype(np.int64)
        mi = (wl.uniform(w4.seed, 9_500_000 + c) * w4.n_m).astype(np.int64)
        assert check_decision_cells(w4, env, t_idx, pi, mi) == 2 * k
