"""Discrete-event simulation of pLogP send schedules (independent check of the oracle's formulas).

pLogP semantics used (Section 2 of the paper; the same ones that make Table 1's
Flat Tree equal (P-1) g(m) + L and its Chain equal (P-1)(g(m) + L)): a node has
one send port, busy for g(size) per message it sends; a message whose
transmission starts at time t is available at its receiver at t + g(size) + L;
a node issues its sends in program order, each as soon as the port is free and
the data it depends on has arrived.  Receiving costs the receiver's port the
same gap: reception starts L after the send started, or when the receiver has
finished its previous reception if that is later, and lasts g(size).  In the
paper's Broadcast and Scatter strategies no node ever receives two messages at
once, so this rule never shows there (arrival = t + g(size) + L); it is what
makes a Gather or a Reduce — many senders, one receiver — take the mirrored
strategy's time.

Nothing here uses the closed-form models: a schedule is a list of sends with
dependencies, and the completion time is the latest arrival.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence


@dataclass
class Send:
    src: int
    dst: int
    size: int
    needs: Sequence[int] = field(default_factory=tuple)  # ids of sends that must have ARRIVED at src


def simulate(n_nodes: int, sends: List[Send], g: Callable[[int], float], L: float) -> float:
    """Run the schedule; sends of one node keep their list order. Returns the completion time."""
    queues = [[] for _ in range(n_nodes)]
    for i, s in enumerate(sends):
        queues[s.src].append(i)
    heads = [0] * n_nodes
    port_free = [0.0] * n_nodes
    rx_free = [0.0] * n_nodes
    arrival: List[Optional[float]] = [None] * len(sends)
    remaining = len(sends)
    while remaining:
        # next event = the ready head-of-queue send with the earliest start time
        best = None
        for node in range(n_nodes):
            if heads[node] >= len(queues[node]):
                continue
            i = queues[node][heads[node]]
            if any(arrival[d] is None for d in sends[i].needs):
                continue
            start = max([port_free[node]] + [arrival[d] for d in sends[i].needs])
            if best is None or start < best[0]:
                best = (start, node, i)
        assert best is not None, "schedule deadlocked"
        start, node, i = best
        busy = g(sends[i].size)
        port_free[node] = start + busy
        dst = sends[i].dst
        arrival[i] = max(start + L, rx_free[dst]) + busy
        rx_free[dst] = arrival[i]
        heads[node] += 1
        remaining -= 1
    return max(arrival) if sends else 0.0


# ---------------- schedule builders (tree shapes only; no cost formulas) ----------------

def flat(P: int, m: int) -> List[Send]:
    return [Send(0, d, m) for d in range(1, P)]


def segmented_flat(P: int, s: int, k: int) -> List[Send]:
    return [Send(0, d, s) for d in range(1, P) for _ in range(k)]


def chain(P: int, m: int) -> List[Send]:
    out = []
    for i in range(P - 1):
        out.append(Send(i, i + 1, m, (len(out) - 1,) if i else ()))
    return out


def segmented_chain(P: int, s: int, k: int) -> List[Send]:
    """Each node forwards a segment as soon as that segment has arrived."""
    out: List[Send] = []
    idx = {}
    for i in range(P - 1):
        for c in range(k):
            idx[(i, c)] = len(out)
            out.append(Send(i, i + 1, s, (idx[(i - 1, c)],) if i else ()))
    return out


def chain_rendezvous(P: int, m: int) -> List[Send]:
    """Per hop: 1-byte request, 1-byte reply, then the payload."""
    out: List[Send] = []
    have = None  # id of the send that delivered the payload to the current holder
    for i in range(P - 1):
        req = len(out)
        out.append(Send(i, i + 1, 1, (have,) if have is not None else ()))
        rep = len(out)
        out.append(Send(i + 1, i, 1, (req,)))
        have = len(out)
        out.append(Send(i, i + 1, m, (rep,)))
    return out


def binary_tree(P: int, m: int) -> List[Send]:
    """Complete binary tree in heap order; a parent serves its left child, then its right child."""
    out: List[Send] = []
    got = {0: None}
    for node in range(P):
        for child in (2 * node + 1, 2 * node + 2):
            if child < P:
                got[child] = len(out)
                out.append(Send(node, child, m, (got[node],) if got[node] is not None else ()))
    return out


def _binomial_edges(P: int):
    """(parent, child, subtree_size_of_child) in each parent's send order, largest subtree first."""
    edges = []

    def cover(lo: int, n: int):
        while n > 1:
            half = 1
            while half * 2 < n:
                half *= 2
            edges.append((lo, lo + half, n - half))
            sub.append((lo + half, n - half))
            n = half

    sub = [(0, P)]
    while sub:
        lo, n = sub.pop(0)
        cover(lo, n)
    return edges


def _tree_schedule(edges, size_of: Callable[[int], int], k: int = 1) -> List[Send]:
    """Each edge carries k messages; a child forwards only after all k have arrived."""
    per_parent = {}
    for e in edges:
        per_parent.setdefault(e[0], []).append(e)  # keeps each parent's own send order
    out: List[Send] = []
    got = {}
    frontier = [0]
    n_edges = 0
    while frontier:
        node = frontier.pop(0)
        for (p, c, n) in per_parent.get(node, []):
            need = (got[p],) if p in got else ()
            for _ in range(k):
                last = len(out)
                out.append(Send(p, c, size_of(n), need))
            got[c] = last
            frontier.append(c)
            n_edges += 1
    assert n_edges == len(edges)
    return out


def binomial(P: int, m: int) -> List[Send]:
    return _tree_schedule(_binomial_edges(P), lambda n: m)


def segmented_binomial(P: int, s: int, k: int) -> List[Send]:
    return _tree_schedule(_binomial_edges(P), lambda n: s, k)


def scatter_flat(P: int, m: int) -> List[Send]:
    return flat(P, m)


def scatter_chain(P: int, m: int) -> List[Send]:
    """Node i passes on the data of everybody behind it: (P-1-i) blocks of m."""
    out = []
    for i in range(P - 1):
        out.append(Send(i, i + 1, (P - 1 - i) * m, (len(out) - 1,) if i else ()))
    return out


def scatter_binomial(P: int, m: int) -> List[Send]:
    """A child receives its own block and those of its whole subtree."""
    return _tree_schedule(_binomial_edges(P), lambda n: n * m)


# ---------------- the mirrored collectives: many senders, one receiver ----------------

def _reversed_tree(edges, size_of: Callable[[int], int], k: int = 1) -> List[Send]:
    """Every edge (parent, child, subtree size) carries k messages from the child to the parent; a child sends
    only after all messages of all its own children have arrived (the mirror image of _tree_schedule)."""
    children = {}
    for (p, c, n) in edges:
        children.setdefault(p, []).append((c, n))
    out: List[Send] = []

    def emit(node: int) -> List[int]:
        """Schedules the subtree below node; returns the ids of the sends that arrive at node."""
        incoming: List[int] = []
        for (c, n) in reversed(children.get(node, [])):   # smallest subtree first: the reverse of the send order
            below = emit(c)
            for _ in range(k):
                incoming.append(len(out))
                out.append(Send(c, node, size_of(n), tuple(below)))
        return incoming

    emit(0)
    return out


def _flat_edges(P: int):
    return [(0, d, 1) for d in range(1, P)]


def gather_flat(P: int, m: int) -> List[Send]:
    return _reversed_tree(_flat_edges(P), lambda n: m)


def gather_chain(P: int, m: int) -> List[Send]:
    """Node i passes on its own block and those of everybody behind it: (P-i) blocks of m."""
    out: List[Send] = []
    for i in range(P - 1, 0, -1):
        out.append(Send(i, i - 1, (P - i) * m, (len(out) - 1,) if i < P - 1 else ()))
    return out


def gather_binomial(P: int, m: int) -> List[Send]:
    return _reversed_tree(_binomial_edges(P), lambda n: n * m)


def reduce_flat(P: int, m: int) -> List[Send]:
    return _reversed_tree(_flat_edges(P), lambda n: m)


def reduce_segmented_flat(P: int, s: int, k: int) -> List[Send]:
    return _reversed_tree(_flat_edges(P), lambda n: s, k)


def reduce_chain(P: int, m: int) -> List[Send]:
    out: List[Send] = []
    for i in range(P - 1, 0, -1):
        out.append(Send(i, i - 1, m, (len(out) - 1,) if i < P - 1 else ()))
    return out


def reduce_segmented_chain(P: int, s: int, k: int) -> List[Send]:
    """Each node passes a segment on as soon as that segment has arrived from behind."""
    out: List[Send] = []
    idx = {}
    for i in range(P - 1, 0, -1):
        for c in range(k):
            idx[(i, c)] = len(out)
            out.append(Send(i, i - 1, s, (idx[(i + 1, c)],) if i < P - 1 else ()))
    return out


def reduce_binomial(P: int, m: int) -> List[Send]:
    return _reversed_tree(_binomial_edges(P), lambda n: m)


def reduce_segmented_binomial(P: int, s: int, k: int) -> List[Send]:
    return _reversed_tree(_binomial_edges(P), lambda n: s, k)


def _binary_edges(P: int):
    return [(node, child, 1) for node in range(P) for child in (2 * node + 1, 2 * node + 2) if child < P]


def reduce_binary(P: int, m: int) -> List[Send]:
    return _reversed_tree(_binary_edges(P), lambda n: m)


def barrier(P: int, up: List[Send], down: List[Send]) -> List[Send]:
    """A reduction of one-byte messages (up) followed by a broadcast of one-byte messages (down): the root's first
    broadcast sends wait for everything that arrives at the root."""
    last = tuple(i for i, snd in enumerate(up) if snd.dst == 0)
    off = len(up)
    shifted = [Send(snd.src, snd.dst, snd.size, tuple(d + off for d in snd.needs) + (last if snd.src == 0 else ())) for snd in down]
    return list(up) + shifted
