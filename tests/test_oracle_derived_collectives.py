"""Pins of the oracle's derived collectives (Gather, Reduce, Barrier: ids 13..26).  The paper prints no model for
them; the oracle derives them as mirrored Scatter / Broadcast strategies and as a Reduce + Broadcast of one-byte
messages.  Here each is compared with the discrete-event simulation of its own send schedule (many senders, one
receiver; the receiver's port pays the gap), never with the mirrored formula."""
import numpy as np
import pytest

import des
from oracle import plogp_oracle as po
from paper_cs_0408034_b200 import workloads as wl

REL = 1e-12


def tables():
    out = []
    for seed in (1, 2, 3):
        sizes = wl.log_spaced_multiples(4, 1 << 16, 10)
        sizes[0] = 1   # the one-byte messages of the Barrier then sit on a breakpoint
        out.append(po.Table(sizes, wl.noisy_monotone_gaps(sizes, 2.0 + seed, 0.02 * seed, 0.1, seed), 3.0 * seed))
    return out


def sim(t, P, sends):
    return des.simulate(P, sends, lambda x: po.gap(t, x), t.L)


def test_gather_equals_its_simulated_schedule():
    for t in tables():
        for P in range(2, 17):
            for m in (4, 96, 2048):
                assert sim(t, P, des.gather_flat(P, m)) == pytest.approx(po.model(t, 13, P, m), rel=REL)
                assert sim(t, P, des.gather_chain(P, m)) == pytest.approx(po.model(t, 14, P, m), rel=REL)
        for P in (2, 4, 8, 16):
            for m in (4, 96, 2048):
                assert sim(t, P, des.gather_binomial(P, m)) == pytest.approx(po.model(t, 15, P, m), rel=REL)


def test_reduce_equals_its_simulated_schedule():
    for t in tables():
        for P in range(2, 17):
            for m in (64, 1024):
                assert sim(t, P, des.reduce_flat(P, m)) == pytest.approx(po.model(t, 16, P, m), rel=REL)
                assert sim(t, P, des.reduce_chain(P, m)) == pytest.approx(po.model(t, 18, P, m), rel=REL)
                assert sim(t, P, des.reduce_binary(P, m)) <= po.model(t, 20, P, m) * (1 + REL)   # printed as a bound
                for s in (16, 64):
                    k = po.segments(m, s)
                    assert sim(t, P, des.reduce_segmented_flat(P, s, k)) == pytest.approx(po.model(t, 17, P, m, s), rel=REL)
                    assert sim(t, P, des.reduce_segmented_chain(P, s, k)) == pytest.approx(po.model(t, 19, P, m, s), rel=REL)
        for P in (2, 4, 8, 16):
            for m in (64, 1024):
                assert sim(t, P, des.reduce_binomial(P, m)) == pytest.approx(po.model(t, 21, P, m), rel=REL)
                for s in (16, 64):
                    k = po.segments(m, s)
                    assert sim(t, P, des.reduce_segmented_binomial(P, s, k)) == pytest.approx(po.model(t, 22, P, m, s), rel=REL)


def test_barrier_equals_reduce_then_broadcast_of_one_byte_messages():
    for t in tables():
        for P in range(2, 17):
            assert sim(t, P, des.barrier(P, des.reduce_flat(P, 1), des.flat(P, 1))) == pytest.approx(po.model(t, 23, P, 4), rel=REL)
            assert sim(t, P, des.barrier(P, des.reduce_chain(P, 1), des.chain(P, 1))) == pytest.approx(po.model(t, 24, P, 4), rel=REL)
            assert sim(t, P, des.barrier(P, des.reduce_binary(P, 1), des.binary_tree(P, 1))) <= po.model(t, 25, P, 4) * (1 + REL)
        for P in (2, 4, 8, 16):
            assert sim(t, P, des.barrier(P, des.reduce_binomial(P, 1), des.binomial(P, 1))) == pytest.approx(po.model(t, 26, P, 4), rel=REL)
        # the message size plays no part in a Barrier
        assert po.model(t, 26, 9, 4) == po.model(t, 26, 9, 1 << 20)


def test_receive_port_rule_on_a_hand_made_schedule():
    g = lambda size: {1: 2.0, 8: 5.0}[size]
    # three senders, one receiver: receptions queue up behind each other, 5 each, the first one starting at L = 3
    assert des.simulate(4, [des.Send(1, 0, 8), des.Send(2, 0, 8), des.Send(3, 0, 8)], g, 3.0) == 3.0 + 3 * 5.0
    # one sender, three receivers: unchanged by the rule (the sender's port paces the messages)
    assert des.simulate(4, [des.Send(0, 1, 8), des.Send(0, 2, 8), des.Send(0, 3, 8)], g, 3.0) == 3 * 5.0 + 3.0


def test_selection_over_the_derived_collectives():
    t = tables()[1]
    sg = po.SGrid([16, 64, 256])
    full = (1 << po.N_STRATEGIES) - 1
    everything = (1 << 27) - 1
    P = [2, 3, 9, 40, 64]
    m = [64, 1000, 1 << 14]
    scatter = po.select_grid(full, po.predict_grid(t, full, P, m, sg))
    gather = po.decide_grid(t, po.GATHER, everything, P, m, sg)
    # a Gather decision is the Scatter decision with the mirrored ids
    assert np.array_equal(gather.strategy, scatter.strategy[1] + 3) and np.array_equal(gather.time, scatter.time[1])
    reduce = po.decide_grid(t, po.REDUCE, everything, P, m, sg)
    no_rdv = full & ~((1 << 1) | (1 << 4) | (1 << 8))
    bcast = po.select_grid(no_rdv, po.predict_grid(t, no_rdv, P, m, sg))
    relabel = {0: 16, 2: 17, 3: 18, 5: 19, 6: 20, 7: 21, 9: 22}
    assert np.array_equal(reduce.strategy, np.vectorize(relabel.get)(bcast.strategy[0]))
    assert np.array_equal(reduce.time, bcast.time[0]) and np.array_equal(reduce.s, bcast.s[0])
    barrier = po.decide_grid(t, po.BARRIER, everything, P, [4], sg)
    for ip, Pv in enumerate(P):
        times = [po.model(t, i, Pv, 4) for i in range(23, 27)]
        assert barrier.time[ip, 0] == min(times) and barrier.strategy[ip, 0] == 23 + int(np.argmin(times))
