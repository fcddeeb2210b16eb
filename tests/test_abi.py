"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

from paper_2409_12490_b200 import binding as cp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "critiprefill.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(critiprefill_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2409_12490_b200.build import build
    build()
    lib = cp.load_library()
    names = declared_symbols()
    assert set(cp.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_params_struct_size_matches_header_layout():
    # 10 int32 + 12 int64 + 3 float + 1 int32
    assert ctypes.sizeof(cp.CpParams) == 10 * 4 + 12 * 8 + 3 * 4 + 4


def test_host_validation_without_gpu():
    p = cp.Problem(1, 4, 2, 1024, 64, 128, 32, 8)
    assert cp.workspace_bytes(p) > 256
    with pytest.raises(cp.CritiPrefillError):
        cp.workspace_bytes(cp.Problem(1, 4, 3, 1024, 64, 128, 32, 8))      # Hq % Hkv
    with pytest.raises(cp.CritiPrefillError):
        cp.workspace_bytes(cp.Problem(1, 4, 2, 1024, 64, 128, 48, 8))      # seg % blk
    with pytest.raises(cp.CritiPrefillError):
        cp.workspace_bytes(cp.Problem(1, 4, 2, 1024, 64, 128, 32, 3))      # k < r
    assert cp.workspace_bytes(cp.Problem(1, 4, 2, 1000, 64, 128, 32, 8)) > 256   # a ragged length is fine
    assert "workspace" in cp.status_string(4)


def test_varlen_sizes_and_cu_seqlens_validation_without_gpu():
    lib = cp.load_library()
    prob = cp.Problem(1, 4, 2, 1000, 64, 128, 32, 8)
    p = prob.params()
    out = [ctypes.c_int64(0) for _ in range(3)]

    def sizes(cu, params=p):
        arr = (ctypes.c_int32 * len(cu))(*cu)
        return lib.critiprefill_varlen_sizes(ctypes.byref(params), arr, len(cu) - 1, *[ctypes.byref(o) for o in out])

    assert sizes([0, 1000, 1300, 1301]) == cp.CP_OK
    n1 = [8, 3, 1]; n2 = [32, 10, 1]
    assert out[0].value == 4 * sum(a * b for a, b in zip(n1, n2))
    assert out[1].value == 4 * sum(n1) * 8 and out[2].value == 4 * sum(n1)
    for bad in ([1, 10], [0, 10, 10], [0, 10, 5], [0, 1001]):        # start, empty, decreasing, longer than seq_len
        assert sizes(bad) == cp.CP_ERR_SHAPE
    p2 = cp.Problem(2, 4, 2, 1000, 64, 128, 32, 8).params()
    assert sizes([0, 10], p2) == cp.CP_ERR_SHAPE                       # a packed batch has batch = 1
