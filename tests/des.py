"""Discrete-event simulation of pLogP send schedules (independent check of the oracle's formulas).

pLogP semantics used (Section 2 of the paper; the same ones that make Table 1's
Flat Tree equal (P-1) g(m) + L and its Chain equal (P-1)(g(m) + L)): a node has
one send port, busy for g(size) per message it sends; a message whose
transmission starts at time t is available at its receiver at t + g(size) + L;
receiving is free; a node issues its sends in program order, each as soon as
the port is free and the data it depends on has arrived.

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
        arrival[i] = start + busy + L
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
