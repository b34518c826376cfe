"""The oracle's Table 1 / Table 2 formulas against a discrete-event simulation of each strategy's
send schedule under pLogP semantics, for tiny process counts and random small tables."""
import numpy as np
import pytest

import des
from oracle import plogp_oracle as po
from paper_cs_0408034_b200 import workloads as wl


def tables():
    out = []
    for seed in range(3):
        sizes = wl.log_spaced_multiples(4, 1 << 14, 8)
        gaps = wl.noisy_monotone_gaps(sizes, 2.0 + seed, 0.02, 0.25, 100 + seed)
        out.append(po.Table(sizes, gaps, 3.0 + 4.0 * seed))
    return out


TABLES = tables()
MS = [8, 96, 1000, 5000]
REL = 1e-11  # the simulation adds up to ~2e4 gaps one by one; a wrong term is off by >1e-3


def sim(t, P, sends):
    return des.simulate(P, sends, lambda x: po.gap(t, x), t.L)


@pytest.mark.parametrize("ti", range(len(TABLES)))
def test_equalities_for_every_P(ti):
    t = TABLES[ti]
    for P in range(2, 17):
        for m in MS:
            assert sim(t, P, des.flat(P, m)) == pytest.approx(po.model(t, 0, P, m), rel=REL)
            assert sim(t, P, des.chain(P, m)) == pytest.approx(po.model(t, 3, P, m), rel=REL)
            assert sim(t, P, des.chain_rendezvous(P, m)) == pytest.approx(po.model(t, 4, P, m), rel=REL)
            assert sim(t, P, des.scatter_flat(P, m)) == pytest.approx(po.model(t, 10, P, m), rel=REL)
            assert sim(t, P, des.scatter_chain(P, m)) == pytest.approx(po.model(t, 11, P, m), rel=REL)
            for s in (4, 8, 32, 96):
                if s > m:
                    continue
                for k_mode in (0, 1):
                    k = po.segments(m, s, k_mode)
                    assert sim(t, P, des.segmented_flat(P, s, k)) == pytest.approx(po.model(t, 2, P, m, s, k_mode), rel=REL)
                    assert sim(t, P, des.segmented_chain(P, s, k)) == pytest.approx(po.model(t, 5, P, m, s, k_mode), rel=REL)


@pytest.mark.parametrize("ti", range(len(TABLES)))
def test_binomial_trees_at_powers_of_two(ti):
    t = TABLES[ti]
    for P in (2, 4, 8, 16):
        for m in MS:
            assert sim(t, P, des.binomial(P, m)) == pytest.approx(po.model(t, 7, P, m), rel=REL)
            assert sim(t, P, des.scatter_binomial(P, m)) == pytest.approx(po.model(t, 12, P, m), rel=REL)
            for s in (4, 32):
                if s <= m:
                    k = po.segments(m, s, 0)
                    assert sim(t, P, des.segmented_binomial(P, s, k)) == pytest.approx(po.model(t, 9, P, m, s), rel=REL)


@pytest.mark.parametrize("ti", range(len(TABLES)))
def test_rendezvous_variants_with_two_processes(ti):
    t = TABLES[ti]
    for m in MS:
        hop = sim(t, 2, des.chain_rendezvous(2, m))
        assert hop == pytest.approx(po.model(t, 1, 2, m), rel=REL)
        assert hop == pytest.approx(po.model(t, 8, 2, m), rel=REL)


@pytest.mark.parametrize("ti", range(len(TABLES)))
def test_bounds_where_the_printed_model_is_not_a_schedule(ti):
    t = TABLES[ti]
    for P in range(2, 17):
        f, c = 1 << po.log2_floor(P), 1 << po.log2_ceil(P)
        for m in MS:
            # Binary Tree is printed as an upper bound
            assert sim(t, P, des.binary_tree(P, m)) <= po.model(t, 6, P, m) * (1 + REL)
            # Binomial trees off the powers of two: simulation and printed value share a bracket
            for sid, sched in ((7, des.binomial(P, m)), (12, des.scatter_binomial(P, m))):
                lo, hi = po.model(t, sid, f, m), po.model(t, sid, c, m)
                got = sim(t, P, sched)
                assert lo * (1 - REL) <= got <= hi * (1 + REL), (sid, P, m)
                assert lo * (1 - REL) <= po.model(t, sid, P, m) <= hi * (1 + REL)


def test_simulator_on_a_hand_schedule():
    # two sends from one port then a dependent forward: 0->1 (g=2), 0->2 (g=2), 1->3 after arrival
    g = lambda x: 2.0
    sends = [des.Send(0, 1, 1), des.Send(0, 2, 1), des.Send(1, 3, 1, (0,))]
    # arrivals: 2+5=7, 4+5=9, 7+2+5=14
    assert des.simulate(4, sends, g, 5.0) == 14.0
