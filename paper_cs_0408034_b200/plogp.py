"""Python binding of the C ABI in ``include/plogp.h`` (same names, argument marshalling only).

Every step of the evaluation runs in the CUDA library; torch is used for device memory and the
current stream.  There is no fallback: if the shared object is missing, importing this module
raises, and the calls need a CUDA device.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libplogp.so")

N_STRATEGIES = 13
SEGMENTED_IDS = (2, 5, 9)
EXPORTS = ("plogp_table_load", "plogp_table_update", "plogp_table_free", "plogp_predict", "plogp_select_best", "plogp_select_best_host",
           "plogp_status_string", "plogp_last_cuda_error", "plogp_kernel_launches", "plogp_fp64_fma_rate", "plogp_profile_enable", "plogp_profile_read",
           "plogp_scatter_chain_static", "plogp_segment_surface", "plogp_segment_sensitivity", "plogp_decision_boundaries",
           "plogp_select_best_collective")

OK, E_INVAL, E_NOMEM, E_CUDA, E_RANGE = 0, -1, -2, -3, -4


class Grid(C.Structure):
    """Mirror of ``plogp_grid``."""
    _fields_ = [("P", C.POINTER(C.c_int32)), ("n_P", C.c_int32), ("P_lo", C.c_int32), ("P_hi", C.c_int32),
                ("m", C.POINTER(C.c_uint64)), ("n_m", C.c_int32),
                ("s", C.POINTER(C.c_uint64)), ("n_s", C.c_int64),
                ("s_lo", C.c_uint64), ("s_hi", C.c_uint64), ("s_step", C.c_uint64),
                ("dtype_bytes", C.c_uint32), ("strategy_mask", C.c_uint32), ("k_mode", C.c_int32),
                ("search_mode", C.c_int32)]


if not os.path.exists(LIB_PATH):
    raise ImportError("%s is missing: build it with `python __graft_entry__.py` (nvcc, sm_100a); "
                      "there is no CPU fallback" % LIB_PATH)
lib = C.CDLL(LIB_PATH)
for _name in EXPORTS:
    if not hasattr(lib, _name):
        raise ImportError("%s does not export %s" % (LIB_PATH, _name))

lib.plogp_table_load.restype = C.c_int
lib.plogp_table_load.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                 C.POINTER(C.c_void_p)]
lib.plogp_table_update.restype = C.c_int
lib.plogp_table_update.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_table_free.restype = C.c_int
lib.plogp_table_free.argtypes = [C.c_void_p]
lib.plogp_predict.restype = C.c_int
lib.plogp_predict.argtypes = [C.c_void_p, C.POINTER(Grid), C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_select_best.restype = C.c_int
lib.plogp_select_best.argtypes = [C.c_void_p, C.POINTER(Grid), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_select_best_host.restype = C.c_int
lib.plogp_select_best_host.argtypes = [C.c_void_p, C.POINTER(Grid), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_status_string.restype = C.c_char_p
lib.plogp_status_string.argtypes = [C.c_int]
lib.plogp_last_cuda_error.restype = C.c_char_p
lib.plogp_last_cuda_error.argtypes = []
lib.plogp_scatter_chain_static.restype = C.c_int
lib.plogp_scatter_chain_static.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_double, C.c_int32, C.c_int32,
                                           C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
lib.plogp_segment_surface.restype = C.c_int
lib.plogp_segment_surface.argtypes = [C.c_void_p, C.POINTER(Grid), C.c_void_p, C.c_void_p]
lib.plogp_segment_sensitivity.restype = C.c_int
lib.plogp_segment_sensitivity.argtypes = [C.c_void_p, C.POINTER(Grid), C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_decision_boundaries.restype = C.c_int
lib.plogp_decision_boundaries.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_select_best_collective.restype = C.c_int
lib.plogp_select_best_collective.argtypes = [C.c_void_p, C.POINTER(Grid), C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.plogp_profile_enable.restype = C.c_int
lib.plogp_profile_enable.argtypes = [C.c_void_p, C.c_int]
lib.plogp_profile_read.restype = C.c_int
lib.plogp_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int32)]
lib.plogp_kernel_launches.restype = C.c_uint64
lib.plogp_kernel_launches.argtypes = []
lib.plogp_fp64_fma_rate.restype = C.c_double
lib.plogp_fp64_fma_rate.argtypes = [C.c_double]


class PlogpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = "%s: %s" % (where, lib.plogp_status_string(status).decode())
        if status == E_CUDA:
            msg += " [%s]" % lib.plogp_last_cuda_error().decode()
        super().__init__(msg)


def _check(status: int, where: str) -> None:
    if status != OK:
        raise PlogpError(status, where)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


class Tables:
    """Owner of a ``plogp_tables`` handle (pLogP parameter sets on the current device)."""

    def __init__(self, sizes, gaps, latency):
        sizes = np.ascontiguousarray(sizes, dtype=np.uint64)
        gaps = np.ascontiguousarray(gaps, dtype=np.float64)
        latency = np.ascontiguousarray(latency, dtype=np.float64)
        if gaps.ndim != 2 or latency.shape != (gaps.shape[0],):
            raise ValueError("gaps must be [n_tables][n_bp] and latency [n_tables]")
        shared = sizes.ndim == 1
        if sizes.shape != (gaps.shape[1],) and sizes.shape != gaps.shape:
            raise ValueError("sizes must be [n_bp] or [n_tables][n_bp]")
        self.n_tables, self.n_bp = int(gaps.shape[0]), int(gaps.shape[1])
        h = C.c_void_p()
        _check(lib.plogp_table_load(self.n_tables, self.n_bp, _ptr(sizes), int(shared), _ptr(gaps),
                                    _ptr(latency), C.byref(h)), "plogp_table_load")
        self._h = h

    @classmethod
    def from_workload(cls, w) -> "Tables":
        return cls(w.sizes, w.gaps, w.latency)

    def update(self, sizes, gaps, latency, stream=None) -> None:
        """``plogp_table_update``: new contents for all tables (same shapes), no reallocation."""
        sizes = np.ascontiguousarray(sizes, dtype=np.uint64)
        gaps = np.ascontiguousarray(gaps, dtype=np.float64)
        latency = np.ascontiguousarray(latency, dtype=np.float64)
        if gaps.shape != (self.n_tables, self.n_bp) or latency.shape != (self.n_tables,):
            raise ValueError("shapes must match the loaded tables")
        if sizes.shape != (self.n_bp,) and sizes.shape != gaps.shape:
            raise ValueError("sizes must be [n_bp] or [n_tables][n_bp]")
        _check(lib.plogp_table_update(self.handle, _ptr(sizes), int(sizes.ndim == 1), _ptr(gaps), _ptr(latency),
                                      _stream_ptr(stream)), "plogp_table_update")

    @property
    def handle(self):
        if self._h is None:
            raise ValueError("tables were freed")
        return self._h

    def free(self) -> None:
        if getattr(self, "_h", None) is not None:
            h, self._h = self._h, None
            _check(lib.plogp_table_free(h), "plogp_table_free")

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.free()

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class GridArgs:
    """Keeps the host arrays of a ``plogp_grid`` alive next to the struct."""

    def __init__(self, m, P=None, P_lo=2, P_hi=2, s=None, s_lo=0, s_hi=0, s_step=0,
                 dtype_bytes=4, strategy_mask=(1 << 13) - 1, k_mode=0, search_mode=0):
        self.m = np.ascontiguousarray(m, dtype=np.uint64)
        self.P = None if P is None else np.ascontiguousarray(P, dtype=np.int32)
        self.s = None if s is None else np.ascontiguousarray(s, dtype=np.uint64)
        g = Grid()
        if self.P is not None:
            g.P = self.P.ctypes.data_as(C.POINTER(C.c_int32))
            g.n_P = len(self.P)
        g.P_lo, g.P_hi = int(P_lo), int(P_hi)
        g.m = self.m.ctypes.data_as(C.POINTER(C.c_uint64))
        g.n_m = len(self.m)
        if self.s is not None:
            g.s = self.s.ctypes.data_as(C.POINTER(C.c_uint64))
            g.n_s = len(self.s)
        g.s_lo, g.s_hi, g.s_step = int(s_lo), int(s_hi), int(s_step)
        g.dtype_bytes, g.strategy_mask, g.k_mode = int(dtype_bytes), int(strategy_mask), int(k_mode)
        g.search_mode = int(search_mode)
        self.struct = g

    @classmethod
    def from_workload(cls, w) -> "GridArgs":
        return cls(w.m, getattr(w, "P_list", None), w.P_lo, w.P_hi, w.s_list, w.s_lo, w.s_hi, w.s_step, w.dtype_bytes,
                   w.strategy_mask, w.k_mode, getattr(w, "search_mode", 0))

    @property
    def n_P(self) -> int:
        return len(self.P) if self.P is not None else self.struct.P_hi - self.struct.P_lo + 1

    @property
    def n_m(self) -> int:
        return len(self.m)

    @property
    def ref(self):
        return C.byref(self.struct)


def _as_grid(grid) -> GridArgs:
    return grid if isinstance(grid, GridArgs) else GridArgs.from_workload(grid)


def _stream_ptr(stream) -> int:
    import torch
    st = torch.cuda.current_stream() if stream is None else stream
    return int(st.cuda_stream)


@dataclass
class Prediction:
    time: "object"    # torch.float64 [n_tables][13][n_P][n_m]
    best_s: "object"  # torch.int32 (uint32 bit pattern) [n_tables][3][n_P][n_m]


@dataclass
class DecisionTable:
    strategy: "object"  # torch.uint8 [n_tables][2][n_P][n_m]
    s_bytes: "object"   # torch.int32 (uint32 bit pattern) [n_tables][2][n_P][n_m]
    time: "object"      # torch.float64 [n_tables][2][n_P][n_m]


def predict(tables: Tables, grid, out: Optional[Prediction] = None, stream=None, want_best_s: bool = True) -> Prediction:
    """``plogp_predict``: all enabled models of Table 1 / Table 2, segmented ones reduced over s."""
    import torch
    g = _as_grid(grid)
    if out is None:
        shape = (tables.n_tables, N_STRATEGIES, g.n_P, g.n_m)
        time = torch.full(shape, float("nan"), dtype=torch.float64, device="cuda")
        best = torch.zeros((tables.n_tables, 3, g.n_P, g.n_m), dtype=torch.int32, device="cuda") if want_best_s else None
        out = Prediction(time, best)
    _check(lib.plogp_predict(tables.handle, g.ref, out.time.data_ptr(),
                             None if out.best_s is None else out.best_s.data_ptr(), _stream_ptr(stream)),
           "plogp_predict")
    return out


def alloc_decision(n_tables: int, n_P: int, n_m: int) -> DecisionTable:
    import torch
    shape = (n_tables, 2, n_P, n_m)
    return DecisionTable(torch.full(shape, 255, dtype=torch.uint8, device="cuda"),
                         torch.zeros(shape, dtype=torch.int32, device="cuda"),
                         torch.full(shape, float("nan"), dtype=torch.float64, device="cuda"))


def select_best(tables: Tables, grid, out: Optional[DecisionTable] = None, stream=None) -> DecisionTable:
    """``plogp_select_best``: best strategy, its segment size and predicted time per (collective, P, m)."""
    g = _as_grid(grid)
    if out is None:
        out = alloc_decision(tables.n_tables, g.n_P, g.n_m)
    _check(lib.plogp_select_best(tables.handle, g.ref, out.strategy.data_ptr(), out.s_bytes.data_ptr(),
                                 out.time.data_ptr(), _stream_ptr(stream)), "plogp_select_best")
    return out


def fp64_fma_rate(milliseconds: float = 50.0) -> float:
    """``plogp_fp64_fma_rate``: sustained thread-level DFMA instructions per second on this device."""
    r = lib.plogp_fp64_fma_rate(float(milliseconds))
    if r < 0:
        raise PlogpError(int(r), "plogp_fp64_fma_rate")
    return r


def kernel_launches() -> int:
    """``plogp_kernel_launches``: kernels launched by the library in this process so far."""
    return int(lib.plogp_kernel_launches())


def scatter_chain_static(d_sizes, d_gap, latency: float, P_lo: int, P_hi: int, d_m, out=None, stream=None):
    """``plogp_scatter_chain_static``: Scatter Chain times [n_P][n_m] for one table, with every
    array already on the device (torch int64 sizes / message sizes, float64 gaps).  The library
    allocates nothing in this call; ``out`` is allocated here, by torch, only when not given."""
    import torch
    if out is None:
        out = torch.empty((P_hi - P_lo + 1, d_m.numel()), dtype=torch.float64, device=d_m.device)
    _check(lib.plogp_scatter_chain_static(int(d_sizes.numel()), d_sizes.data_ptr(), d_gap.data_ptr(), float(latency),
                                          int(P_lo), int(P_hi), d_m.data_ptr(), int(d_m.numel()), out.data_ptr(),
                                          _stream_ptr(stream)), "plogp_scatter_chain_static")
    return out


KERNEL_KINDS = ("sweep_kernel", "s1_tile_sum_kernel", "fused_kernel", "decide_kernel", "scatter_kernel", "envelope_kernel", "segmin_kernel", "gaps_kernel")


def profile_enable(tables: Tables, enable: bool = True) -> None:
    """``plogp_profile_enable``: record CUDA events around every kernel launched on this handle."""
    _check(lib.plogp_profile_enable(tables.handle, int(enable)), "plogp_profile_enable")


def profile_read(tables: Tables) -> dict:
    """``plogp_profile_read``: {kernel kind: (milliseconds, launches)} since the last read."""
    ms = (C.c_double * len(KERNEL_KINDS))()
    n = (C.c_int32 * len(KERNEL_KINDS))()
    _check(lib.plogp_profile_read(tables.handle, ms, n), "plogp_profile_read")
    return {k: (ms[i], n[i]) for i, k in enumerate(KERNEL_KINDS) if n[i]}


def alloc_decision_host(n_tables: int, n_P: int, n_m: int) -> DecisionTable:
    """Page-locked host arrays shaped like a decision table (for ``select_best_host``)."""
    import torch
    shape = (n_tables, 2, n_P, n_m)
    return DecisionTable(torch.empty(shape, dtype=torch.uint8, pin_memory=True),
                         torch.empty(shape, dtype=torch.int32, pin_memory=True),
                         torch.empty(shape, dtype=torch.float64, pin_memory=True))


def select_best_host(tables: Tables, grid, out: Optional[DecisionTable] = None, stream=None) -> DecisionTable:
    """``plogp_select_best_host``: the decision table delivered into host arrays (returns when complete)."""
    g = _as_grid(grid)
    if out is None:
        out = alloc_decision_host(tables.n_tables, g.n_P, g.n_m)
    _check(lib.plogp_select_best_host(tables.handle, g.ref, out.strategy.data_ptr(), out.s_bytes.data_ptr(),
                                      out.time.data_ptr(), _stream_ptr(stream)), "plogp_select_best_host")
    return out


def n_candidates(grid) -> int:
    """Number of candidate segment sizes of a grid (the last dimension of the surface)."""
    g = _as_grid(grid)
    if g.s is not None:
        return len(g.s)
    st = g.struct
    return 0 if st.s_step == 0 or st.s_hi < st.s_lo else int((st.s_hi - st.s_lo) // st.s_step) + 1


def segment_surface(tables: Tables, grid, out=None, stream=None):
    """``plogp_segment_surface``: models of ids 2, 5, 9 for every candidate s, [n_tables][3][n_P][n_m][n_s]."""
    import torch
    g = _as_grid(grid)
    if out is None:
        out = torch.full((tables.n_tables, 3, g.n_P, g.n_m, n_candidates(g)), float("inf"), dtype=torch.float64, device="cuda")
    _check(lib.plogp_segment_surface(tables.handle, g.ref, out.data_ptr(), _stream_ptr(stream)), "plogp_segment_surface")
    return out


def segment_sensitivity(tables: Tables, grid, s_fixed: int, pred: Optional[Prediction] = None, stream=None):
    """``plogp_segment_sensitivity``: (time with the fixed segment size, its ratio to the searched minimum), each
    [n_tables][3][n_P][n_m]; the ratio is None when no prediction is given."""
    import torch
    g = _as_grid(grid)
    shape = (tables.n_tables, 3, g.n_P, g.n_m)
    fixed = torch.full(shape, float("nan"), dtype=torch.float64, device="cuda")
    ratio = None if pred is None else torch.full(shape, float("nan"), dtype=torch.float64, device="cuda")
    _check(lib.plogp_segment_sensitivity(tables.handle, g.ref, int(s_fixed), None if pred is None else pred.time.data_ptr(),
                                         fixed.data_ptr(), None if ratio is None else ratio.data_ptr(), _stream_ptr(stream)),
           "plogp_segment_sensitivity")
    return fixed, ratio


def decision_boundaries(dec: DecisionTable, stream=None):
    """``plogp_decision_boundaries``: uint8 flags [n_tables][2][n_P][n_m] (bit 0: changes with P, bit 1: with m)."""
    import torch
    n_tables, _, n_P, n_m = dec.strategy.shape
    out = torch.empty_like(dec.strategy)
    _check(lib.plogp_decision_boundaries(n_tables, n_P, n_m, dec.strategy.data_ptr(), out.data_ptr(), _stream_ptr(stream)),
           "plogp_decision_boundaries")
    return out


GATHER, REDUCE, BARRIER = 2, 3, 4


def select_best_collective(tables: Tables, grid, collective: int, stream=None) -> DecisionTable:
    """``plogp_select_best_collective``: decision table of a derived collective (GATHER, REDUCE: [n_tables][n_P][n_m];
    BARRIER: [n_tables][n_P])."""
    import torch
    g = _as_grid(grid)
    shape = (tables.n_tables, g.n_P) if collective == BARRIER else (tables.n_tables, g.n_P, g.n_m)
    out = DecisionTable(torch.full(shape, 255, dtype=torch.uint8, device="cuda"),
                        torch.zeros(shape, dtype=torch.int32, device="cuda"),
                        torch.full(shape, float("nan"), dtype=torch.float64, device="cuda"))
    _check(lib.plogp_select_best_collective(tables.handle, g.ref, int(collective), out.strategy.data_ptr(), out.s_bytes.data_ptr(),
                                            out.time.data_ptr(), _stream_ptr(stream)), "plogp_select_best_collective")
    return out
