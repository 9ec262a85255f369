"""The C-ABI library builds for sm_100a, loads without a GPU and exports what the header declares."""
import ctypes
import os
import re

from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "actkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(actkv_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_calls():
    names = _declared()
    for f in ("actkv_score", "actkv_select", "actkv_compact", "actkv_budget"):
        assert f in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build_mod.build()
    lib = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(lib, name), name
    assert set(B.EXPORTS) <= set(_declared())
    assert b"sm_100a" in ctypes.cast(lib.actkv_version, ctypes.CFUNCTYPE(ctypes.c_char_p))()


def test_workspace_queries_run_without_a_gpu():
    lib = B.load()
    assert lib.actkv_compact_workspace_bytes(8, 2188) >= 4 * (2 * 8 + 8 * 2188)
    assert lib.actkv_select_workspace_bytes(192, 8, 35000) >= 0
    assert lib.actkv_budget_workspace_bytes(512, 8, 4096) >= 512 * 4 + 8 * 4096 * 4
    pd = B.PoolDesc(1, 48, 1000, 16, 4, 128, 0, 0, 0, 0, 0)
    assert B.actkv_score_workspace_bytes(pd, 8, 48, 32, 512, 64, 35000) > 0


def test_binding_refuses_cpu_tensors():
    import pytest
    import torch
    with pytest.raises(TypeError):
        B.actkv_keep_indptr(torch.zeros(2, dtype=torch.int32), torch.zeros(2, dtype=torch.int32), 2,
                            torch.zeros(3, dtype=torch.int32))


def test_host_side_checks_of_the_newer_entry_points_run_without_a_gpu():
    import ctypes as C
    lib = B.load()
    pd = B.PoolDesc(1, 48, 1000, 16, 4, 128, 1, 1, 1, 1, 1)
    base = lib.actkv_compact_workspace_bytes(8, 2188)
    d1 = B.actkv_compact_deferred_workspace_bytes(pd, 8, 2188, 1, 9100)
    d16 = B.actkv_compact_deferred_workspace_bytes(pd, 8, 2188, 16, 9100)
    # base + one 32-entry table row per item: ceil(9100 / 16) pages x 8 requests x layers x (16 x 4 / 32) parts
    assert d1 >= base + 569 * 8 * 2 * 128 and d16 >= base + 16 * 569 * 8 * 2 * 128 and d16 < base + 17 * 569 * 8 * 2 * 128 + 4096
    # the fault-injection hook validates its arguments on the host
    assert lib.actkv_debug_inject_stall(3, 0) == B.E_INVALID
    assert lib.actkv_debug_inject_stall(-1, 0) == 0
    # null descriptors are refused before anything is launched
    null = C.c_void_p(None)
    assert lib.actkv_compact_begin(None, None, 0, 1, null, 0, null, null, 0, 0, null, 0, null, null) == B.E_INVALID
    assert lib.actkv_compact_end(None, None, 0, 1, null, 0, null, null, 0, null, 0, null, null) == B.E_INVALID
    assert lib.actkv_compact_stats(null, null, null) == B.E_INVALID
    assert lib.actkv_score_path(None, 32, 64, 0.1, null, 0) == B.E_INVALID
