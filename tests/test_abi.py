"""The C-ABI library loads without a GPU and exports every symbol include/hos.h declares."""
import ctypes as C
import os
import re

import paper_2502_15763_b200 as hos

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hos.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hos_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = hos.lib()
    names = declared_symbols()
    assert set(hos.exported_symbols()) == set(names)
    for n in names:
        assert getattr(L, n) is not None, n


def test_strerror_and_host_side_validation():
    assert hos.hos_strerror(0) == "ok"
    assert "workspace" in hos.hos_strerror(-2)
    L = hos.lib()
    # null batch is rejected on the host, before any CUDA call
    assert L.hos_offline_pack(None, None, 0, None, None, None, None, None, None, None, None, C.c_size_t(0), None) == -1
    assert L.hos_lower_bound(None, None, None, None, None, C.c_size_t(0), None) == -1
    assert L.hos_online_workspace_bytes(None, 1, 0) == 0


def test_struct_sizes_match_the_header():
    assert hos.LS_MOVE_DTYPE.itemsize == 24
    assert hos.LB_DTYPE.itemsize == 72
    assert hos.CLIENT_RESULT_DTYPE.itemsize == 40
    assert hos.SIM_RESULT_DTYPE.itemsize == 32
    assert hos.ITER_REC_DTYPE.itemsize == 16
