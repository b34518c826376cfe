"""Seeded synthetic pLogP workloads (tables + evaluation grids).

Input generation only: this module draws gap tables and builds the (P, m, s)
grids of the five benchmark configurations.  It contains none of the cost-model
arithmetic and is the only module that both the CUDA path's callers and the CPU
oracle's callers use.

The tables stand in for the measured pLogP parameters of Section 2 of the paper
(a gap g(m) at a list of message sizes plus a latency L); configuration 1 copies
the paper's network class (switched 100 Mbit/s Ethernet = 0.08 us per byte).

Random numbers come from a counter-based SplitMix64: u(seed, c) is the top 53
bits of mix(seed + (c + 1) * 0x9E3779B97F4A7C15), so any element can be drawn
independently of the others.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

ALL_STRATEGIES = (1 << 13) - 1
BASE_SEED = 408034 * 10


def uniform(seed: int, counters) -> np.ndarray:
    """u(seed, c) in [0, 1) for every counter c (vectorised SplitMix64 finaliser)."""
    c = np.asarray(counters, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = np.uint64(seed) + (c + np.uint64(1)) * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return (z >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def log_uniform(lo: float, hi: float, u) -> np.ndarray:
    return lo * (hi / lo) ** np.asarray(u, dtype=np.float64)


def log_spaced_multiples(lo: int, hi: int, n: int, multiple: int = 4) -> np.ndarray:
    """n sizes from lo to hi, log-spaced, rounded to the nearest multiple and forced strictly increasing."""
    i = np.arange(n, dtype=np.float64)
    raw = lo * (hi / lo) ** (i / (n - 1)) if n > 1 else np.array([float(lo)])
    x = (np.rint(raw / multiple) * multiple).astype(np.int64)
    x = np.maximum(x, multiple)
    for k in range(1, n):
        if x[k] <= x[k - 1]:
            x[k] = x[k - 1] + multiple
    return x.astype(np.uint64)


def noisy_monotone_gaps(sizes, overhead, per_byte, eps, seed, counter_base=0) -> np.ndarray:
    """g_i = (overhead + per_byte * size_i) * (1 + eps * (2u_i - 1)), then running maximum."""
    sizes = np.asarray(sizes, dtype=np.float64)
    u = uniform(seed, counter_base + np.arange(len(sizes)))
    g = (overhead + per_byte * sizes) * (1.0 + eps * (2.0 * u - 1.0))
    return np.maximum.accumulate(g)


@dataclass
class Workload:
    """Tables plus grid, in the form the library's entry points take them."""
    name: str
    sizes: np.ndarray            # uint64 [n_bp] (shared) or [n_tables][n_bp]
    gaps: np.ndarray             # float64 [n_tables][n_bp]
    latency: np.ndarray          # float64 [n_tables]
    P_lo: int
    P_hi: int
    m: np.ndarray                # uint64 [n_m], ascending multiples of dtype_bytes
    s_list: Optional[np.ndarray] = None   # uint64 ascending; None => s_lo..s_hi step s_step
    s_lo: int = 0
    s_hi: int = 0
    s_step: int = 0
    strategy_mask: int = ALL_STRATEGIES
    k_mode: int = 0
    dtype_bytes: int = 4
    seed: int = 0
    notes: dict = field(default_factory=dict)
    P_list: Optional[np.ndarray] = None   # int32 ascending process counts; None => P_lo..P_hi
    search_mode: int = 0                  # 0 = exhaustive segment search, 1 = lower envelope (same results)

    @property
    def n_tables(self) -> int:
        return int(self.gaps.shape[0])

    @property
    def n_bp(self) -> int:
        return int(self.gaps.shape[1])

    @property
    def sizes_shared(self) -> bool:
        return self.sizes.ndim == 1

    @property
    def n_P(self) -> int:
        return len(self.P_list) if self.P_list is not None else self.P_hi - self.P_lo + 1

    @property
    def n_m(self) -> int:
        return len(self.m)

    def P_values(self) -> np.ndarray:
        if self.P_list is not None:
            return np.asarray(self.P_list, dtype=np.int64)
        return np.arange(self.P_lo, self.P_hi + 1, dtype=np.int64)

    def s_values(self) -> np.ndarray:
        if self.s_list is not None:
            return self.s_list
        return np.arange(self.s_lo, self.s_hi + 1, self.s_step, dtype=np.uint64)

    def table_sizes(self, t: int) -> np.ndarray:
        return self.sizes if self.sizes_shared else self.sizes[t]

    def n_candidates(self) -> np.ndarray:
        """Per message size: how many grid segment sizes fit (s <= m), at least 1 (unsegmented fallback)."""
        if self.s_list is not None:
            c = np.searchsorted(self.s_list, self.m, side="right")
        else:
            top = np.minimum(self.m.astype(np.int64), self.s_hi)
            c = np.where(top >= self.s_lo, (top - self.s_lo) // self.s_step + 1, 0)
        return np.maximum(c, 1).astype(np.int64)

    def model_cells(self) -> int:
        """(table, strategy, P, m[, s]) formula evaluations in one pass; Scatter Chain counts one per (P, m)."""
        mask = self.strategy_mask
        n_seg = sum((mask >> b) & 1 for b in (2, 5, 9))
        n_unseg = sum((mask >> b) & 1 for b in range(13)) - n_seg
        per_table = self.n_P * (n_seg * int(self.n_candidates().sum()) + n_unseg * self.n_m)
        return per_table * self.n_tables

    def decision_cells(self) -> int:
        mask = self.strategy_mask
        n_coll = int(bool(mask & 0x3FF)) + int(bool(mask & 0x1C00))
        return self.n_tables * n_coll * self.n_P * self.n_m


def _bits(*ids) -> int:
    return sum(1 << i for i in ids)


def config1() -> Workload:
    """Ethernet-like single table (100 Mbit/s, as the paper's cluster), P = 2..50, power-of-two m and s."""
    seed = BASE_SEED + 1
    sizes = (2 ** np.arange(21)).astype(np.uint64)
    gaps = noisy_monotone_gaps(sizes, 30.0, 0.08, 0.02, seed)[None, :]
    return Workload("cfg1_ethernet_P50", sizes, gaps, np.array([50.0]), 2, 50,
                    (2 ** np.arange(2, 21)).astype(np.uint64),
                    s_list=(2 ** np.arange(10, 17)).astype(np.uint64),
                    strategy_mask=_bits(0, 3, 5, 6, 7, 10, 11, 12), seed=seed)


def config2(P_hi: int = 1024, n_m: int = 256, n_s: int = 64) -> Workload:
    """Dense grid on one table of the configuration-1 generator; all 13 strategies."""
    seed = BASE_SEED + 2
    sizes = (2 ** np.arange(21)).astype(np.uint64)
    gaps = noisy_monotone_gaps(sizes, 30.0, 0.08, 0.02, seed)[None, :]
    return Workload("cfg2_dense_P%d" % P_hi, sizes, gaps, np.array([50.0]), 2, P_hi,
                    log_spaced_multiples(4, 64 << 20, n_m),
                    s_list=log_spaced_multiples(4, 1 << 20, n_s), seed=seed)


def config3(P_hi: int = 4096, n_m: int = 128, m_lo: int = 4 << 10, m_hi: int = 16 << 20,
            s_hi: int = 1 << 20) -> Workload:
    """Exhaustive segment sweep: every multiple of 4 B up to min(m, 1 MB); segmented flat + segmented chain."""
    seed = BASE_SEED + 3
    sizes = log_spaced_multiples(4, 16 << 20, 64)
    gaps = noisy_monotone_gaps(sizes, 1.0, 0.0008, 0.01, seed)[None, :]
    return Workload("cfg3_sweep_P%d" % P_hi, sizes, gaps, np.array([5.0]), 2, P_hi,
                    log_spaced_multiples(m_lo, m_hi, n_m), s_lo=4, s_hi=s_hi, s_step=4,
                    strategy_mask=_bits(2, 5), seed=seed)


def config4(n_tables: int = 4096, P_hi: int = 512, n_m: int = 128, n_s: int = 32,
            seed_offset: int = 0) -> Workload:
    """Batched multi-network tuning: independent tables with log-uniform latency, bandwidth and overhead."""
    seed = BASE_SEED + 4 + seed_offset
    sizes = log_spaced_multiples(4, 256 << 20, 64)
    t = np.arange(n_tables, dtype=np.uint64)
    base = t << np.uint64(20)
    latency = log_uniform(1.0, 100.0, uniform(seed, base + np.uint64(1000)))
    rate_bits_per_us = log_uniform(100.0, 400000.0, uniform(seed, base + np.uint64(1001)))
    per_byte = 8.0 / rate_bits_per_us
    overhead = log_uniform(0.5, 50.0, uniform(seed, base + np.uint64(1002)))
    u = uniform(seed, base[:, None] + np.arange(64, dtype=np.uint64)[None, :])
    g = (overhead[:, None] + per_byte[:, None] * sizes.astype(np.float64)[None, :]) * (1.0 + 0.03 * (2.0 * u - 1.0))
    gaps = np.maximum.accumulate(g, axis=1)
    return Workload("cfg4_batched_T%d" % n_tables, sizes, np.ascontiguousarray(gaps), latency, 2, P_hi,
                    log_spaced_multiples(4, 64 << 20, n_m),
                    s_list=log_spaced_multiples(4, 1 << 20, n_s), seed=seed)


def config5(P_hi: int = 65536, n_m: int = 64) -> Workload:
    """Scatter-heavy long sums: chain and binomial Scatter (flat kept so a decision exists), P up to 65536."""
    seed = BASE_SEED + 5
    sizes = log_spaced_multiples(4, 256 << 20, 128)
    gaps = noisy_monotone_gaps(sizes, 1.0, 0.00004, 0.01, seed)[None, :]
    return Workload("cfg5_scatter_P%d" % P_hi, sizes, gaps, np.array([2.0]), 2, P_hi,
                    log_spaced_multiples(4, 4 << 10, n_m), s_list=None, s_lo=4, s_hi=4, s_step=4,
                    strategy_mask=_bits(10, 11, 12), seed=seed)


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def shard_tables(w: Workload, rank: int, world: int) -> Workload:
    """Contiguous slice of the tables for one rank (tables are independent problems)."""
    T = w.n_tables
    lo = (T * rank) // world
    hi = (T * (rank + 1)) // world
    sizes = w.sizes if w.sizes_shared else w.sizes[lo:hi]
    return replace(w, name="%s_r%dof%d" % (w.name, rank, world), sizes=sizes,
                   gaps=np.ascontiguousarray(w.gaps[lo:hi]), latency=np.ascontiguousarray(w.latency[lo:hi]))
