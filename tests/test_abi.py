"""The C-ABI library loads without a GPU and exports every function the public header declares (no compute calls)."""
import ctypes as C
import os
import re

from paper_2609_03079_b200 import binding as ls
from paper_2609_03079_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(?:int32_t|int64_t|size_t)\s+(ls_\w+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = C.CDLL(path)
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert sorted(ls.EXPORTS) == names  # the Python binding covers the same names


def test_struct_layouts_match_the_header():
    lib = ls.lib()
    d = ls.ls_layer_desc()
    d.struct_size = C.sizeof(ls.ls_layer_desc) - 4
    out = C.c_void_p()
    assert lib.ls_layer_create(C.byref(d), C.byref(out)) == ls.LS_ERR_INVALID
    assert str(C.sizeof(ls.ls_layer_desc)) in ls.last_error()  # the library expects exactly the ctypes size
    assert out.value is None


def test_host_side_argument_checks_without_a_gpu():
    lib = ls.lib()
    assert lib.ls_layer_destroy(None) == ls.LS_OK
    assert lib.ls_layer_create(None, None) == ls.LS_ERR_INVALID
    assert "NULL" in ls.last_error()
    sel = ls.ls_selection()
    assert lib.ls_predict(None, None, 1, 1, C.byref(sel), None) == ls.LS_ERR_INVALID
    assert lib.ls_cache_stats(None, None) == ls.LS_ERR_INVALID
    assert ls.ls_version() == 1000 and ls.ls_kernel_launches() == 0
    n, ms = C.c_int64(7), C.c_double(1.0)
    assert lib.ls_timing_read(0, C.byref(n), C.byref(ms)) == ls.LS_OK and n.value == 0 and ms.value == 0.0
