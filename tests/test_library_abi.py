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
