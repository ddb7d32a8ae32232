"""The C-ABI library loads and exports every symbol include/dg.h declares (CPU only)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2104_06700_b200 import build
    return build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dg_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_call_list():
    names = declared_symbols()
    for required in ("dg_graph_create", "dg_graph_transpose", "dg_aggregate_fwd",
                     "dg_aggregate_bwd", "dg_graph_destroy"):
        assert required in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} is declared in dg.h but not exported"


def test_binding_lists_the_same_symbols(libpath):
    from paper_2104_06700_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    assert binding.dg_version().startswith("libdgagg")


def test_host_side_argument_checks_need_no_gpu(libpath):
    """Checks that fail before any CUDA call: they must return a status, never crash."""
    lib = ctypes.CDLL(libpath)
    lib.dg_last_error.restype = ctypes.c_char_p
    h = ctypes.c_void_p()
    i64 = ctypes.c_int64
    assert lib.dg_graph_create(i64(4), i64(2), None, None, None, None) == 1   # out_graph NULL
    assert lib.dg_graph_create(i64(-1), i64(0), None, None, None, ctypes.byref(h)) == 1
    assert lib.dg_graph_create(i64(1 << 31), i64(0), None, None, None, ctypes.byref(h)) == 2
    assert lib.dg_graph_create(i64(4), i64(2), None, None, None, ctypes.byref(h)) == 1
    assert b"rowptr" in lib.dg_last_error()
    assert lib.dg_graph_destroy(None) == 0
    assert lib.dg_aggregate_fwd(None, None, 4, 0, None, None) == 1
    assert lib.dg_aggregate_bwd(None, None, 4, 0, None, None) == 1
    assert lib.dg_graph_transpose(None, None, 0, None, 0, None) == 1
    assert lib.dg_graph_validate(None, None) == 1


def test_product_path_has_no_oracle_import():
    pkg = os.path.join(ROOT, "paper_2104_06700_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f
                assert "ap_oracle" not in src, f
