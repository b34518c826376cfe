"""The shared library loads without a GPU and exports every symbol that include/plogp.h declares."""
import ctypes
import os
import re

import __graft_entry__ as ge

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "plogp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(plogp_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_the_header():
    ge.build()
    from paper_cs_0408034_b200 import plogp
    lib = ctypes.CDLL(plogp.LIB_PATH)
    syms = declared_symbols()
    assert {"plogp_table_load", "plogp_table_free", "plogp_predict", "plogp_select_best",
            "plogp_status_string"} <= set(syms)
    for name in syms:
        assert hasattr(lib, name), name
    assert set(plogp.EXPORTS) == set(syms)


def test_status_strings_need_no_device():
    from paper_cs_0408034_b200 import plogp
    assert plogp.lib.plogp_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4):
        assert plogp.lib.plogp_status_string(code) not in (b"ok", b"unknown status")
    assert plogp.lib.plogp_status_string(-99) == b"unknown status"


def test_grid_struct_matches_the_header_layout(tmp_path):
    """sizeof / offsetof as gcc sees the header must equal the ctypes mirror."""
    import subprocess
    from paper_cs_0408034_b200 import plogp
    fields = [f for f, _ in plogp.Grid._fields_]
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "plogp.h"\nint main(void){printf("%zu", sizeof(plogp_grid));'
                   + "".join('printf(" %%zu", offsetof(plogp_grid, %s));' % f for f in fields) + "return 0;}\n")
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert got[0] == ctypes.sizeof(plogp.Grid)
    assert got[1:] == [getattr(plogp.Grid, f).offset for f in fields]


def test_table_validation_runs_on_the_host_before_any_device_call():
    """Malformed tables are refused with a status code without touching CUDA (works without a GPU)."""
    import numpy as np
    from paper_cs_0408034_b200 import plogp

    def status(sizes, gaps, lat, shared=1):
        sizes = np.ascontiguousarray(sizes, dtype=np.uint64)
        gaps = np.ascontiguousarray(gaps, dtype=np.float64)
        lat = np.ascontiguousarray(lat, dtype=np.float64)
        h = ctypes.c_void_p()
        rc = plogp.lib.plogp_table_load(gaps.shape[0], gaps.shape[1], sizes.ctypes.data, shared, gaps.ctypes.data,
                                        lat.ctypes.data, ctypes.byref(h))
        assert h.value is None or rc == 0
        if rc == 0:
            plogp.lib.plogp_table_free(h)
        return rc

    assert status([4, 4, 16], [[1.0, 2.0, 3.0]], [1.0]) == plogp.E_INVAL
    assert status([4, 8, 16], [[1.0, float("nan"), 3.0]], [1.0]) == plogp.E_INVAL
    assert status([4, 8, 16], [[1.0, 2.0, 3.0]], [-1.0]) == plogp.E_INVAL
    assert status([4], [[1.0]], [1.0]) == plogp.E_INVAL
    assert status([4, 8, 1 << 60], [[1.0, 2.0, 3.0]], [1.0]) == plogp.E_RANGE
    assert status([4, 8, 16], [[1.0, 3.0, 2.0]], [1.0]) == plogp.E_RANGE   # falling last interval: g would turn negative above the table
    assert status([4, 8, 16], [[1.0, 3.0, 2.0]], [float("inf")]) == plogp.E_INVAL
    assert status([[4, 8, 16], [4, 8, 8]], [[1.0, 2.0, 3.0], [1.0, 2.0, 3.0]], [1.0, 1.0], shared=0) == plogp.E_INVAL
    h = ctypes.c_void_p()
    assert plogp.lib.plogp_table_load(1, 3, None, 1, None, None, ctypes.byref(h)) == plogp.E_INVAL
    assert plogp.lib.plogp_select_best(None, None, None, None, None, None) == plogp.E_INVAL
    assert plogp.lib.plogp_predict(None, None, None, None, None) == plogp.E_INVAL
    assert plogp.lib.plogp_scatter_chain_static(8, None, None, 1.0, 2, 3, None, 1, None, None) == plogp.E_INVAL
    assert plogp.lib.plogp_table_free(None) == plogp.OK
