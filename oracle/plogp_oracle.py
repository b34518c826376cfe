"""ctypes front end of the CPU oracle (``plogp_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is a plain host evaluator of the paper's
Table 1 / Table 2 cost models, the Section 3.1 segment-size search and the
strategy selection; it shares nothing with the CUDA library and must never be
imported by the product path.  Only the tests, the smoke check and the
CPU-baseline leg of the benchmark use it.

This module does argument marshalling only; every number comes from the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "plogp_oracle.c")
_HDR = os.path.join(_HERE, "plogp_oracle.h")
_LIB = os.path.join(_HERE, "libplogp_oracle.so")

N_STRATEGIES = 13
SEGMENTED_IDS = (2, 5, 9)
STRATEGY_NAMES = (
    "bcast_flat", "bcast_flat_rdv", "bcast_seg_flat", "bcast_chain", "bcast_chain_rdv",
    "bcast_seg_chain", "bcast_binary", "bcast_binomial", "bcast_binomial_rdv",
    "bcast_seg_binomial", "scatter_flat", "scatter_chain", "scatter_binomial",
)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) into a shared object next to its source."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.run(["gcc", "-std=c99", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall",
                        "-ffp-contract=off", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Table(C.Structure):
    _fields_ = [("n_bp", C.c_int), ("size", C.POINTER(C.c_uint64)),
                ("gap", C.POINTER(C.c_double)), ("L", C.c_double)]


class _SGrid(C.Structure):
    _fields_ = [("list", C.POINTER(C.c_uint64)), ("n_list", C.c_int64),
                ("lo", C.c_uint64), ("hi", C.c_uint64), ("step", C.c_uint64)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        TP, SP = C.POINTER(_Table), C.POINTER(_SGrid)
        lib.po_gap.restype = C.c_double
        lib.po_gap.argtypes = [TP, C.c_uint64]
        lib.po_log2_floor.argtypes = [C.c_int64]
        lib.po_log2_ceil.argtypes = [C.c_int64]
        lib.po_segments.restype = C.c_uint64
        lib.po_segments.argtypes = [C.c_uint64, C.c_uint64, C.c_int]
        lib.po_model.restype = C.c_double
        lib.po_model.argtypes = [TP, C.c_int, C.c_int64, C.c_uint64, C.c_uint64, C.c_int]
        lib.po_segment_search.restype = None
        lib.po_segment_search.argtypes = [TP, C.c_int, C.c_int64, C.c_uint64, SP, C.c_int,
                                          C.POINTER(C.c_uint64), C.POINTER(C.c_double),
                                          C.POINTER(C.c_double)]
        lib.po_decide.argtypes = [TP, C.c_int, C.c_uint32, C.c_int64, C.c_uint64, SP, C.c_int,
                                  C.POINTER(C.c_int), C.POINTER(C.c_uint64),
                                  C.POINTER(C.c_double), C.POINTER(C.c_double)]
        lib.po_predict_grid.restype = None
        lib.po_predict_grid.argtypes = [TP, C.c_uint32, C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                        SP, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.po_select_grid.restype = None
        lib.po_select_grid.argtypes = [C.c_uint32, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.po_effective_segment.restype = C.c_uint64
        lib.po_effective_segment.argtypes = [C.c_uint64, C.c_uint64]
        lib.po_surface_grid.restype = None
        lib.po_surface_grid.argtypes = [TP, C.c_uint32, C.c_void_p, C.c_int, C.c_void_p, C.c_int, SP, C.c_int, C.c_void_p]
        lib.po_fixed_segment_grid.restype = None
        lib.po_fixed_segment_grid.argtypes = [TP, C.c_uint32, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_uint64,
                                              C.c_int, C.c_void_p]
        lib.po_decide_grid.restype = None
        lib.po_decide_grid.argtypes = [TP, C.c_int, C.c_uint32, C.c_void_p, C.c_int, C.c_void_p, C.c_int, SP, C.c_int,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.po_threads.restype = C.c_int
        _lib = lib
    return _lib


class Table:
    """One pLogP parameter set: sizes (bytes, strictly increasing), gaps, latency L."""

    def __init__(self, sizes, gaps, L):
        self.sizes = np.ascontiguousarray(sizes, dtype=np.uint64)
        self.gaps = np.ascontiguousarray(gaps, dtype=np.float64)
        assert self.sizes.ndim == 1 and self.sizes.shape == self.gaps.shape and len(self.sizes) >= 2
        self.L = float(L)
        self._c = _Table(len(self.sizes), self.sizes.ctypes.data_as(C.POINTER(C.c_uint64)),
                         self.gaps.ctypes.data_as(C.POINTER(C.c_double)), self.L)

    @property
    def ref(self):
        return C.byref(self._c)


class SGrid:
    """Candidate segment sizes: explicit ascending list, or every lo + i*step <= hi."""

    def __init__(self, values=None, lo=0, hi=0, step=0):
        if values is not None:
            self.values = np.ascontiguousarray(values, dtype=np.uint64)
            self._c = _SGrid(self.values.ctypes.data_as(C.POINTER(C.c_uint64)), len(self.values), 0, 0, 0)
        else:
            self.values = None
            self._c = _SGrid(None, 0, int(lo), int(hi), int(step))

    @property
    def ref(self):
        return C.byref(self._c)


def threads() -> int:
    return _load().po_threads()


def gap(t: Table, x: int) -> float:
    return _load().po_gap(t.ref, int(x))


def log2_floor(P: int) -> int:
    return _load().po_log2_floor(int(P))


def log2_ceil(P: int) -> int:
    return _load().po_log2_ceil(int(P))


def segments(m: int, s: int, k_mode: int = 0) -> int:
    return _load().po_segments(int(m), int(s), int(k_mode))


def model(t: Table, strategy: int, P: int, m: int, s: int = 0, k_mode: int = 0) -> float:
    return _load().po_model(t.ref, int(strategy), int(P), int(m), int(s), int(k_mode))


def segment_search(t: Table, strategy: int, P: int, m: int, sg: SGrid, k_mode: int = 0):
    """-> (best_s, best_time, runner_up_time) over the candidates s <= m."""
    s, bt, ru = C.c_uint64(), C.c_double(), C.c_double()
    _load().po_segment_search(t.ref, int(strategy), int(P), int(m), sg.ref, int(k_mode),
                              C.byref(s), C.byref(bt), C.byref(ru))
    return s.value, bt.value, ru.value


def decide(t: Table, collective: int, mask: int, P: int, m: int, sg: SGrid, k_mode: int = 0):
    """-> (strategy, s, time, runner_up_time) or None when nothing is enabled."""
    sid, s, bt, ru = C.c_int(), C.c_uint64(), C.c_double(), C.c_double()
    rc = _load().po_decide(t.ref, int(collective), int(mask), int(P), int(m), sg.ref, int(k_mode),
                           C.byref(sid), C.byref(s), C.byref(bt), C.byref(ru))
    if rc != 0:
        return None
    return sid.value, s.value, bt.value, ru.value


@dataclass
class Predicted:
    time: np.ndarray     # [13][n_P][n_m] float64 (NaN where disabled)
    best_s: np.ndarray   # [3][n_P][n_m] uint64
    seg_runner_up: np.ndarray  # [3][n_P][n_m] float64


@dataclass
class Decision:
    strategy: np.ndarray   # [2][n_P][n_m] uint8
    s: np.ndarray          # [2][n_P][n_m] uint64
    time: np.ndarray       # [2][n_P][n_m] float64
    runner_up: np.ndarray  # [2][n_P][n_m] float64


def predict_grid(t: Table, mask: int, P, m, sg: SGrid, k_mode: int = 0) -> Predicted:
    P = np.ascontiguousarray(P, dtype=np.int64)
    m = np.ascontiguousarray(m, dtype=np.uint64)
    nP, nm = len(P), len(m)
    time = np.full((N_STRATEGIES, nP, nm), np.nan, dtype=np.float64)
    best_s = np.zeros((3, nP, nm), dtype=np.uint64)
    ru = np.full((3, nP, nm), np.inf, dtype=np.float64)
    _load().po_predict_grid(t.ref, int(mask), P.ctypes.data, nP, m.ctypes.data, nm, sg.ref,
                            int(k_mode), time.ctypes.data, best_s.ctypes.data, ru.ctypes.data)
    return Predicted(time, best_s, ru)


def select_grid(mask: int, pred: Predicted) -> Decision:
    _, nP, nm = pred.time.shape
    strategy = np.zeros((2, nP, nm), dtype=np.uint8)
    s = np.zeros((2, nP, nm), dtype=np.uint64)
    time = np.zeros((2, nP, nm), dtype=np.float64)
    ru = np.zeros((2, nP, nm), dtype=np.float64)
    _load().po_select_grid(int(mask), nP, nm, pred.time.ctypes.data, pred.best_s.ctypes.data,
                           strategy.ctypes.data, s.ctypes.data, time.ctypes.data, ru.ctypes.data)
    return Decision(strategy, s, time, ru)


def n_candidates(sg: SGrid) -> int:
    if sg.values is not None:
        return len(sg.values)
    c = sg._c
    return 0 if c.step == 0 or c.hi < c.lo else int((c.hi - c.lo) // c.step) + 1


def surface_grid(t: Table, mask: int, P, m, sg: SGrid, k_mode: int = 0) -> np.ndarray:
    """Model surface over s: [3][n_P][n_m][n_s] for ids 2, 5, 9 (NaN where s > m or the id is disabled)."""
    P = np.ascontiguousarray(P, dtype=np.int64)
    m = np.ascontiguousarray(m, dtype=np.uint64)
    out = np.full((3, len(P), len(m), n_candidates(sg)), np.nan, dtype=np.float64)
    _load().po_surface_grid(t.ref, int(mask), P.ctypes.data, len(P), m.ctypes.data, len(m), sg.ref, int(k_mode),
                            out.ctypes.data)
    return out


def fixed_segment_grid(t: Table, mask: int, P, m, s_fixed: int, k_mode: int = 0) -> np.ndarray:
    """Times of ids 2, 5, 9 with one fixed segment size (the whole message where it does not fit): [3][n_P][n_m]."""
    P = np.ascontiguousarray(P, dtype=np.int64)
    m = np.ascontiguousarray(m, dtype=np.uint64)
    out = np.full((3, len(P), len(m)), np.nan, dtype=np.float64)
    _load().po_fixed_segment_grid(t.ref, int(mask), P.ctypes.data, len(P), m.ctypes.data, len(m), int(s_fixed),
                                  int(k_mode), out.ctypes.data)
    return out


def effective_segment(m: int, s_fixed: int) -> int:
    return _load().po_effective_segment(int(m), int(s_fixed))


def decision_boundaries(strategy: np.ndarray) -> np.ndarray:
    """Where the selected strategy changes in the (P, m) plane: for strategy[..., n_P, n_m] returns uint8 flags of
    the same shape, bit 0 = differs from the next larger P (same m), bit 1 = differs from the next larger m
    (same P); the last row / column has no such neighbour and gets 0 there."""
    s = np.asarray(strategy)
    out = np.zeros(s.shape, dtype=np.uint8)
    out[..., :-1, :] |= (s[..., :-1, :] != s[..., 1:, :]).astype(np.uint8)
    out[..., :, :-1] |= ((s[..., :, :-1] != s[..., :, 1:]).astype(np.uint8) << 1)
    return out


# Collectives the paper names without printing models (derived in plogp_oracle.h): ids and what they mirror
GATHER, REDUCE, BARRIER = 2, 3, 4
DERIVED_FIRST_ID = {GATHER: 13, REDUCE: 16, BARRIER: 23}
MIRROR_OF = {13: 10, 14: 11, 15: 12, 16: 0, 17: 2, 18: 3, 19: 5, 20: 6, 21: 7, 22: 9}   # derived id -> printed id
BARRIER_SHAPE_OF = {23: 0, 24: 3, 25: 6, 26: 7}                                           # barrier id -> tree shape's Broadcast id


def decide_grid(t: Table, collective: int, mask: int, P, m, sg: SGrid, k_mode: int = 0) -> Decision:
    """po_decide for every (P, m): Decision with [n_P][n_m] arrays (strategy 255 where nothing is enabled)."""
    P = np.ascontiguousarray(P, dtype=np.int64)
    m = np.ascontiguousarray(m, dtype=np.uint64)
    nP, nm = len(P), len(m)
    strategy = np.zeros((nP, nm), dtype=np.uint8)
    s = np.zeros((nP, nm), dtype=np.uint64)
    time = np.zeros((nP, nm), dtype=np.float64)
    ru = np.zeros((nP, nm), dtype=np.float64)
    _load().po_decide_grid(t.ref, int(collective), int(mask), P.ctypes.data, nP, m.ctypes.data, nm, sg.ref, int(k_mode),
                           strategy.ctypes.data, s.ctypes.data, time.ctypes.data, ru.ctypes.data)
    return Decision(strategy, s, time, ru)
