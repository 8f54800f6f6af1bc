"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import os
import re

import paper_2608_12146_b200.binding as rp
from paper_2608_12146_b200 import build as rpbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "routepack.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rp_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    path = rpbuild.build()
    assert os.path.exists(path)
    lib = rp.lib()
    names = declared_functions()
    assert {"rp_window_load", "rp_place_experts", "rp_pack_rows", "rp_eval_population", "rp_anneal",
            "rp_best"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(rp.EXPORTS)


def test_strerror_names_every_status():
    lib = rp.lib()
    for code in range(0, -10, -1):
        assert lib.rp_strerror(code).decode() != "unknown status"
    assert lib.rp_strerror(-99).decode() == "unknown status"


def test_null_arguments_are_rejected_without_a_device():
    import ctypes as C
    lib = rp.lib()
    out = C.c_void_p(123)
    assert lib.rp_window_load(C.byref(out), None, None, None, None) == -1 and out.value is None
    assert lib.rp_place_experts(None, None, None) == -1
    assert lib.rp_pack_rows(None, None, None) == -1
    assert lib.rp_anneal(None, None, None) == -1
    assert lib.rp_best(None, None, None, None) == -1
    assert lib.rp_eval_population(None, None, 0, None, None) == -1
    lib.rp_destroy(None)
