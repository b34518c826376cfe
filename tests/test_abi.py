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
