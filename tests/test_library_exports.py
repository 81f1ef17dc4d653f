"""The C-ABI library builds, loads without a GPU and exports every function that
include/ps.h declares.  No compute call is made here."""
import ctypes
import os
import re

from paper_2601_02311_b200 import build as ps_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+char\s*\*|int|void|uint64_t)\s+(ps_[a-z_]+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_header_declares_the_three_entry_points():
    names = declared_functions()
    for required in ("ps_eval_batch", "ps_sweep_pareto", "ps_check_composition"):
        assert required in names
    assert len(names) >= 14


def test_library_builds_and_exports_every_declared_symbol():
    lib_path = ps_build.build()
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), name
    lib.ps_strerror.restype = ctypes.c_char_p
    assert lib.ps_strerror(0) == b"ok"
    assert b"range" in lib.ps_strerror(-3)


def test_binding_lists_the_same_symbols():
    import paper_2601_02311_b200.ps as ps
    assert sorted(ps.EXPORTS) == declared_functions()
